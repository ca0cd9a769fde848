// Expert FFN, tensor-core variant for prefill-sized batches: a persistent grouped GEMM on tcgen05.
//
// Roles inside the MMA: the M dimension (128 lanes of tensor memory) holds weight rows, the N dimension
// holds up to 256 tokens of one expert.  A work item is (expert, pass of <= 256 tokens, tile of 256 weight
// rows); the 256 rows are two M=128 MMAs that share one token stage in shared memory (each token tile read
// from L2 feeds twice the math) and own one 256-column accumulator each: all 512 columns of tensor memory.
// An expert with more than 256 rows is cut into equal passes, so the padding of a ragged expert is at
// most 15 tokens per pass.  For the gate/up stage the first M=128 tile is 128 gate rows and the second the 128
// matching up rows, so gate and up of one i sit in the same tensor-memory lane of the two accumulators.
//
// Warp roles (one CTA per SM, persistent):
//   warp 0       producer: TMA loads of the token tile (bf16, 128-byte swizzle) and of the packed codes
//   warp 1       allocates tensor memory, issues tcgen05.mma (one lane), commits to mbarriers
//   warps 2..9   one thread per weight row: packed E2M1 codes from the TMA-fed packed ring, exact expansion
//                to bf16 scaled by the E8M0 block scale, written into the swizzled K-major A stage the
//                tensor core reads
//   warps 10..17 epilogue, two warps per lane quadrant taking alternate column chunks: tcgen05.ld the
//                accumulators; stage 1 applies SwiGLU thread-locally (gate and up share a lane) and stores bf16
//                pairs; stage 2 stores fp32 rows
// Every mbarrier wait is bounded and reports through the status word.
#include <cuda.h>

#include "moe_sm100_primitives.cuh"

namespace moe {

namespace {

constexpr int kTileRows = 256;    // weight rows per work item: two M=128 MMA tiles
constexpr int kBlockK = 64;       // K per pipeline stage: one 128-byte row of bf16
constexpr int kMaxTok = 256;      // tokens per pass
constexpr int kTokBox = 64;       // token rows per TMA box
constexpr int kStages = 3;        // A/B ring depth
constexpr int kDequantWarps = 8;
constexpr int kEpilogueWarps = 8;
constexpr int kThreadsUmma = (2 + kDequantWarps + kEpilogueWarps) * 32;  // 576
constexpr int kFirstDequantWarp = 2;
constexpr int kFirstEpilogueWarp = 2 + kDequantWarps;  // 10: (warp % 4) = 2,3,0,1 covers the four lane quadrants
constexpr uint32_t kTmemCols = 512;

constexpr int kATile = 128 * kBlockK * 2;            // 16 KB: one M=128 tile of a stage
constexpr int kABytes = 2 * kATile;                  // 32 KB
constexpr int kBBytes = kMaxTok * kBlockK * 2;       // 32 KB
constexpr int kPStages = 4;                          // packed-code ring (one K block per stage)
constexpr int kPBytes = kTileRows * (kBlockK / 2);   // 8 KB: 256 rows x 32 bytes

struct UmmaArgs {
  const uint8_t* w;        // [E, R, K/2] packed codes
  const uint8_t* sc;       // [E, R, K/32] scale bytes (or moe_prepack's tiles of [128 rows][16 bytes])
  int blocked;             // weights in moe_prepack's tile-contiguous layout (see ExpertWeights)
  const int* offsets;      // [E+1]
  __nv_bfloat16* act;      // stage 1 output [S, I]
  float* y;                // stage 2 output [S, R]
  float* const* row_dst;   // or null; else output row p goes to row_dst[p] (see y_row)
  int* status;
  uint32_t k1, k2;         // 0x1040, 0x0104: multipliers of the E2M1 expansion, kept opaque to the compiler
  int E, K, R, I;          // R weight rows per expert (2I or H)
};

struct SmemMap {
  uint32_t a, b, p, bars, misc, prefix, total;
};
__host__ __device__ inline SmemMap smem_map(int E) {
  SmemMap m;
  uint32_t off = 0;
  m.a = off;
  off += kStages * kABytes;
  m.b = off;
  off += kStages * kBBytes;
  m.p = off;
  off += kPStages * kPBytes;
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

// rows [row0, row0 + ntok) of pass `pass` of an expert with rows [r_begin, r_end): equal passes, 16-aligned
MOE_DEVINL void pass_rows(int r_begin, int r_end, int pass, int* row0, int* ntok) {
  const int m = r_end - r_begin;
  const int np = (m + kMaxTok - 1) / kMaxTok;
  const int tp = (((m + np - 1) / np) + 15) & ~15;
  *row0 = r_begin + pass * tp;
  *ntok = min(tp, m - pass * tp);
}

MOE_DEVINL float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

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
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  uint64_t* full_a = bars;                      // [kStages] dequant warps -> MMA
  uint64_t* full_b = bars + kStages;            // [kStages] TMA -> MMA
  uint64_t* empty_ab = bars + 2 * kStages;      // [kStages] MMA done -> producer, dequant warps
  uint64_t* full_p = bars + 3 * kStages;        // [kPStages] TMA -> dequant warps
  uint64_t* empty_p = full_p + kPStages;        // [kPStages] dequant warps -> producer
  uint64_t* acc_full = empty_p + kPStages;      // MMA -> epilogue
  uint64_t* acc_empty = acc_full + 1;           // epilogue -> MMA
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sm.misc);
  int* prefix = reinterpret_cast<int*>(smem + sm.prefix);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int K = a.K;
  const int num_kb = K / kBlockK;
  const int tiles_per_expert = a.R / kTileRows;

  // ---- setup: pass prefix over experts, barriers, tensor memory ----
  if (wid == 2) {
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
    for (int s = 0; s < kPStages; ++s) {
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
    // =========================== producer: token tiles ===========================
    if (lane == 0) {
      int s = 0, ps = 0;
      uint32_t ph = 0, pph = 0;
      for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
        const int g = w / tiles_per_expert, rt = w % tiles_per_expert;
        const int e = find_expert(prefix, a.E, g);
        int row0, ntok;
        pass_rows(a.offsets[e], a.offsets[e + 1], g - prefix[e], &row0, &ntok);
        const int nbox = (ntok + kTokBox - 1) / kTokBox;
        // packed rows of the tile: stage 1 = 128 gate rows then the 128 matching up rows; stage 2 = 256 rows
        const int wrow_a = STAGE1 ? e * a.R + rt * 128 : e * a.R + rt * kTileRows;
        const int wrow_b = STAGE1 ? e * a.R + a.I + rt * 128 : wrow_a + 128;
        for (int kb = 0; kb < num_kb; ++kb) {
          mbar_wait(&empty_p[ps], pph ^ 1u, a.status);
          mbar_expect_tx(&full_p[ps], kPBytes);
          // 128 rows x 32 bytes of codes; tile-contiguous layout: a quarter of the 128-byte rows of tile (row / 128, kb / 4)
          const int wx = a.blocked ? (kb & 3) * (kBlockK / 2) : kb * (kBlockK / 2);
          const int wya = a.blocked ? ((wrow_a >> 7) * (num_kb >> 2) + (kb >> 2)) * 128 : wrow_a;
          const int wyb = a.blocked ? ((wrow_b >> 7) * (num_kb >> 2) + (kb >> 2)) * 128 : wrow_b;
          tma_load_2d(sP + ps * kPBytes, &tmap_w, wx, wya, &full_p[ps]);
          tma_load_2d(sP + ps * kPBytes + kPBytes / 2, &tmap_w, wx, wyb, &full_p[ps]);
          if (++ps == kPStages) { ps = 0; pph ^= 1u; }
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
        int row0, ntok;
        pass_rows(a.offsets[e], a.offsets[e + 1], g - prefix[e], &row0, &ntok);
        const int n16 = (ntok + 15) & ~15;
        const uint32_t idesc = umma_idesc_bf16(128, n16);
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
            const uint64_t bdesc = umma_desc_k_sw128(b_addr + k4 * 32);
            const uint32_t acc = (kb | k4) != 0 ? 1u : 0u;
            umma_bf16(tmem_base, umma_desc_k_sw128(a_addr + k4 * 32), bdesc, idesc, acc);
            umma_bf16(tmem_base + 256, umma_desc_k_sw128(a_addr + kATile + k4 * 32), bdesc, idesc, acc);
          }
          umma_commit(&empty_ab[s]);
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
        umma_commit(acc_full);
        acc_ph ^= 1u;
      }
    }
  } else if (wid < kFirstEpilogueWarp) {
    // =========================== E2M1 -> bf16 expansion, one thread per weight row ===========================
    const int r = tid - kFirstDequantWarp * 32;   // 0..255
    const int t = r >> 7, l = r & 127;            // MMA tile, lane (row) inside it
    int s = 0, ps = 0;
    uint32_t ph = 0, pph = 0;
    for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
      const int g = w / tiles_per_expert, rt = w % tiles_per_expert;
      const int e = find_expert(prefix, a.E, g);
      // stage 1: tile 0 = gate rows rt*128.., tile 1 = the matching up rows; stage 2: 256 consecutive rows
      const int grow = STAGE1 ? e * a.R + t * a.I + rt * 128 + l : e * a.R + rt * kTileRows + r;
      // this row's scale bytes, 16 (= 8 K blocks) per load: K/32 consecutive bytes, or in the tile-contiguous layout
      // its 16 bytes of tile (row / 128, group of 8 K blocks), the tiles of a row block 2 KB apart
      const uint8_t* srow = a.blocked ? a.sc + (static_cast<size_t>(grow >> 7) * (K / 512)) * 2048 + (grow & 127) * 16
                                      : a.sc + static_cast<size_t>(grow) * (K / 32);
      const int sgroup = a.blocked ? 2048 : 16;  // bytes from one group of 8 K blocks to the next
      const int prow = r;  // row of this thread inside the packed stage (stage 1: gate rows 0..127, up rows 128..255)
      // scale bytes: 16 bytes cover 8 K blocks; fetched one group ahead
      uint4 sc_cur = __ldg(reinterpret_cast<const uint4*>(srow));
      uint4 sc_next = sc_cur;
      unsigned char* arow_base = sA + t * kATile + l * 128;
      for (int kb = 0; kb < num_kb; ++kb) {
        if ((kb & 7) == 0) {
          if (kb != 0) sc_cur = sc_next;
          if (kb + 8 < num_kb) sc_next = __ldg(reinterpret_cast<const uint4*>(srow + ((kb + 8) >> 3) * sgroup));
        }
        const int sidx = (kb & 7) >> 1;  // 32-bit word of the 16 scale bytes; two bytes per K block
        const uint32_t sword = (sidx == 0) ? sc_cur.x : (sidx == 1) ? sc_cur.y : (sidx == 2) ? sc_cur.z : sc_cur.w;
        const uint32_t spair = sword >> ((kb & 1) * 16);
        const uint32_t m_lo = scale_mult(spair & 0xFFu), m_hi = scale_mult((spair >> 8) & 0xFFu);
        mbar_wait(&full_p[ps], pph, a.status);
        const uint4 ca = *reinterpret_cast<const uint4*>(sP + ps * kPBytes + prow * 32);
        const uint4 cb = *reinterpret_cast<const uint4*>(sP + ps * kPBytes + prow * 32 + 16);
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_p[ps]);
        if (++ps == kPStages) { ps = 0; pph ^= 1u; }
        const uint32_t wv[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
        uint4 out[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          uint32_t p[4];
          dequant8(wv[q], q < 4 ? m_lo : m_hi, a.k1, a.k2, p);
          // (0,4),(1,5),(2,6),(3,7) -> natural order (0,1),(2,3),(4,5),(6,7)
          out[q].x = __byte_perm(p[0], p[1], 0x5410);
          out[q].y = __byte_perm(p[2], p[3], 0x5410);
          out[q].z = __byte_perm(p[0], p[1], 0x7632);
          out[q].w = __byte_perm(p[2], p[3], 0x7632);
        }
        mbar_wait(&empty_ab[s], ph ^ 1u, a.status);
        unsigned char* arow = arow_base + s * kABytes;
#pragma unroll
        for (int q = 0; q < 8; ++q) *reinterpret_cast<uint4*>(arow + ((q ^ (l & 7)) << 4)) = out[q];
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&full_a[s]);
        if (++s == kStages) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // =========================== epilogue ===========================
    const int q = wid & 3;                                // tensor-memory lane quadrant this warp may read
    const int half = (wid - kFirstEpilogueWarp) >> 2;     // the two warps of a quadrant take alternate column chunks
    const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
    uint32_t acc_ph = 0;
    for (int w = blockIdx.x; w < total_work; w += gridDim.x) {
      const int g = w / tiles_per_expert, rt = w % tiles_per_expert;
      const int e = find_expert(prefix, a.E, g);
      int row0, ntok;
      pass_rows(a.offsets[e], a.offsets[e + 1], g - prefix[e], &row0, &ntok);
      mbar_wait(acc_full, acc_ph, a.status);
      __syncwarp();  // tcgen05.ld is warp-collective
      tc_fence_after_sync();
      if (STAGE1) {
        // lane = i inside the tile: gate in the first accumulator, up in the second, one token per column.
        // Neighbouring lanes swap one value per token pair so that each thread stores a bf16 pair (i, i + 1).
        const int i = rt * 128 + q * 32 + lane;
        const int odd = lane & 1;
#pragma unroll 1
        for (int c0 = half * 16; c0 < ntok; c0 += 32) {
          uint32_t gv[16], uv[16];
          tmem_ld_32x16(tmem_base + lane_base + static_cast<uint32_t>(c0), gv);
          tmem_ld_32x16(tmem_base + lane_base + static_cast<uint32_t>(256 + c0), uv);
          tmem_ld_wait();
#pragma unroll
          for (int jj = 0; jj < 16; jj += 2) {
            const float v0 = silu_mul(__uint_as_float(gv[jj]), __uint_as_float(uv[jj]));          // token c0 + jj
            const float v1 = silu_mul(__uint_as_float(gv[jj + 1]), __uint_as_float(uv[jj + 1]));  // token c0 + jj + 1
            const float got = __shfl_xor_sync(0xffffffffu, odd ? v0 : v1, 1);
            // even lane: token c0 + jj, rows (i, i + 1); odd lane: token c0 + jj + 1, rows (i - 1, i)
            const __nv_bfloat162 o = odd ? __floats2bfloat162_rn(got, v1) : __floats2bfloat162_rn(v0, got);
            const int tok = c0 + jj + odd;
            if (tok < ntok)
              *reinterpret_cast<__nv_bfloat162*>(a.act + static_cast<size_t>(row0 + tok) * a.I + (i & ~1)) = o;
          }
        }
      } else {
#pragma unroll 1
        for (int t = 0; t < 2; ++t) {
          const uint32_t tcol = tmem_base + lane_base + static_cast<uint32_t>(t * 256);
          const int n = rt * kTileRows + t * 128 + q * 32 + lane;
#pragma unroll 1
          for (int c0 = half * 32; c0 < ntok; c0 += 64) {
            uint32_t v[32];
            tmem_ld_32x32(tcol + static_cast<uint32_t>(c0), v);
            tmem_ld_wait();
#pragma unroll
            for (int jj = 0; jj < 32; ++jj)
              if (c0 + jj < ntok) y_row(a.y, a.row_dst, static_cast<size_t>(row0 + c0 + jj), a.R)[n] = __uint_as_float(v[jj]);
          }
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
  // K % 512: a row's scale bytes (K/32 of them) are then 16-byte aligned for the vector prefetch;
  // rows per expert (2I and H) are then whole 256-row tiles
  return sh.H % 512 == 0 && sh.I % 512 == 0 && static_cast<long long>(sh.T) * sh.k >= 1024 &&
         smem_map(sh.E).total + 1024 <= 227 * 1024;
}

int launch_expert_ffn_umma(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& sh,
                           __nv_bfloat16* act, float* y_perm, int* status_word, cudaStream_t st, float* const* row_dst) {
  const size_t smem = smem_map(sh.E).total + 1024;
  static PerDeviceFlag flag;
  if (!once_per_device(flag, [] {
        return cudaFuncSetAttribute(ffn_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess &&
               cudaFuncSetAttribute(ffn_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
      }))
    return MOE_ERR_CUDA;
  const uint64_t S = static_cast<uint64_t>(sh.T) * sh.k;
  CUtensorMap tm_x, tm_act, tm_w13, tm_w2;
  if (!make_map_2d(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x_perm, sh.H, S, kBlockK, kTokBox, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map_2d(&tm_act, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, act, sh.I, S, kBlockK, kTokBox, CU_TENSOR_MAP_SWIZZLE_128B) ||
      // codes: rows of K/2 bytes, or (tile-contiguous layout) tiles of [128 rows][128 bytes] one after the other
      !make_map_2d(&tm_w13, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w.w13, w.blocked ? 128 : sh.H / 2,
                   static_cast<uint64_t>(sh.E) * 2 * sh.I * (w.blocked ? sh.H / 256 : 1), kBlockK / 2, 128,
                   CU_TENSOR_MAP_SWIZZLE_NONE) ||
      !make_map_2d(&tm_w2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w.w2, w.blocked ? 128 : sh.I / 2,
                   static_cast<uint64_t>(sh.E) * sh.H * (w.blocked ? sh.I / 256 : 1), kBlockK / 2, 128, CU_TENSOR_MAP_SWIZZLE_NONE))
    return MOE_ERR_CUDA;
  const int grid = sm_count();
  UmmaArgs a;
  a.offsets = offsets;
  a.act = act;
  a.y = y_perm;
  a.row_dst = row_dst;
  a.status = status_word;
  a.k1 = 0x1040u;
  a.k2 = 0x0104u;
  a.E = sh.E;
  a.I = sh.I;
  a.blocked = w.blocked ? 1 : 0;
  a.w = w.w13;
  a.sc = w.s13;
  a.K = sh.H;
  a.R = 2 * sh.I;
  ffn_umma_kernel<true><<<grid, kThreadsUmma, smem, st>>>(tm_x, tm_w13, a);
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  a.w = w.w2;
  a.sc = w.s2;
  a.K = sh.I;
  a.R = sh.H;
  ffn_umma_kernel<false><<<grid, kThreadsUmma, smem, st>>>(tm_act, tm_w2, a);
  if (cudaGetLastError() != cudaSuccess) return MOE_ERR_CUDA;
  note_kernel("ffn_umma_tcgen05_grouped", 2);
  return MOE_OK;
}

}  // namespace moe
