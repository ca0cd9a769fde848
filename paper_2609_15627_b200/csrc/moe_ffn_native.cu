// Expert FFN for decode-sized batches on the native block-scaled FP4 tensor-core path:
// packed E2M1 codes and E8M0 scales go HBM -> TMA -> shared memory -> tcgen05.mma with no ALU expansion.
//
// tcgen05.mma kind::mxf8f6f4.block_scale multiplies an E4M3 operand by an E2M1 operand with one UE8M0 scale per
// 32 K elements on both sides - the checkpoint format of the expert weights is exactly such an operand.  The
// activations are bf16, so each row is split on the fly into two E4M3 rows with their own block scales,
//   x = 2^s * hi + 2^(s-3) * lo,   hi = e4m3(x / 2^s),   lo = e4m3((x / 2^s - hi) * 8),
// which is exact for every element within 2^14 of its block's maximum (8 significant bits = 4 + 4) and loses
// less than 2^-19 of the block maximum otherwise; products are exact and accumulate in fp32 in tensor memory.
//
// Operand roles: the tensor core walks the M rows of its A operand one per cycle and all N columns in parallel,
// so the weights are the B operand (N = 256 weight rows per MMA, K = 32) and the tokens the A operand (M = 128
// rows of which 16 are used: 8 tokens x {hi, lo}; the other rows read whatever follows in shared memory and
// their accumulator lanes are never looked at).  With the weights on M the MMA rate capped the stream at
// about 3 TB/s.
//
// Work item = (touched expert, tile of 256 weight rows) over the full K (stage 1: 128 gate + 128 up rows, so
// gate and up of the same i are two columns of the same accumulator lane).
// Warp roles (one persistent CTA per SM):
//   warp 0      producer: TMA loads of the weight tile (4-bit tensor map that unpacks to the 16-byte-aligned
//               operand layout, 128-byte swizzle) and of the scale bytes
//   warp 1      allocates tensor memory, issues the MMAs, commits to mbarriers
//   warps 2..5  move weight scale bytes into tensor memory (tcgen05.st), and at an expert change split that
//               expert's token rows into the E4M3 pair and lay them out as the A operand
//   warp 8      epilogue (lane quadrant 0 holds the 16 used rows): hi + lo, SwiGLU + bf16 rounding + re-split
//               for stage 2 (stage 1) or the fp32 store (stage 2)
// Every wait is bounded and reports through the status word.
#include <cuda.h>
#include <cuda_fp8.h>

#include "moe_sm100_primitives.cuh"

namespace moe {

namespace {

constexpr int kTile = 256;            // weight rows per item (N of the MMA)
constexpr int kKStep = 128;           // K elements per stage (one 128-byte swizzled row per weight row)
constexpr int kWStage = kTile * 128;  // 32 KB of shared memory per stage (16 KB of HBM bytes)
constexpr int kWStages = 4;
constexpr int kScStages = 3;          // scale-byte ring: one stage = 256 rows x 16 bytes = 4 K steps
constexpr int kScStage = kTile * 16;
constexpr int kSfGroups = 3;          // tensor-memory groups for the weight scale factors: 4 K steps x 8 columns
constexpr int kMaxTokPass = 8;        // tokens per pass (16 operand rows)
constexpr int kMaxK = 4096;           // activation operand of one expert stays resident: 16 rows x K bytes
constexpr int kNatThreads = 9 * 32;
constexpr int kEpiWarp = 8;           // warp 8: (8 % 4) == 0 -> may read tensor-memory lanes 0..31
constexpr uint32_t kNatTmemCols = 512;
// tensor-memory columns: one 256-column accumulator; 4 columns per K step for the activation scales (a scale-factor
// block covers 128 rows in 4 columns - rows 32c..32c+31 in column c - and must start on a multiple of 4 columns; only
// lanes 0..15 of its first column carry data here); 3 groups of 4 K steps x 8 columns for the weight scales
constexpr uint32_t kColD = 0, kColSfAct = 256, kColSfW = 384;

struct NatArgs {
  const __nv_bfloat16* x;    // stage 1: sorted token rows [S, K]
  const uint8_t* aq;         // stage 2 input / stage 1 output: split activations [2S, I] (row 2p hi, 2p+1 lo)
  const uint8_t* aq_sf;      //   and their scale bytes [2S, I/32]
  uint8_t* aq_out;
  uint8_t* aq_sf_out;
  const int* offsets;
  float* y;                  // stage 2 output [S, R]
  int* status;
  int E, K, R, I;
};

struct NatSmem {
  uint32_t act, w, sc, sfa, bars, misc, touched, total;
};
__host__ __device__ inline NatSmem nat_smem(int E, int K) {
  NatSmem m;
  uint32_t off = 0;
  m.act = off;  // first: an MMA reads 128 operand rows from a 16-row tile, i.e. up to 14 KB past it, into the ring
  off += 16 * static_cast<uint32_t>(K);
  m.w = off;
  off += kWStages * kWStage;
  m.sc = off;
  off += kScStages * kScStage;
  m.sfa = off;
  off += 16 * (static_cast<uint32_t>(K) / 32);
  m.bars = off;
  off += 64 * 8;
  m.misc = off;
  off += 64;
  m.touched = off;
  off += (static_cast<uint32_t>(E) + 8) * 4;
  m.total = off;
  return m;
}

MOE_DEVINL void tmem_st_32x4(uint32_t taddr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};" ::"r"(taddr), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
               : "memory");
}
MOE_DEVINL void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem, E4M3] * B[smem, E2M1]^T with UE8M0 block scales held in tensor memory
MOE_DEVINL void umma_mxf4(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa, uint32_t sfb,
                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
      :
      : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
      : "memory");
}
// instruction descriptor: A E4M3, B E2M1, UE8M0 scales, M = 128, N = 256; `j` picks byte j of the scale words
MOE_DEVINL uint32_t idesc_mxf4(uint32_t j) {
  return (0u << 7) | (5u << 10) | ((256u >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24) | (j << 29) | (j << 4);
}

MOE_DEVINL float e4m3_to_float(uint32_t byte) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw(static_cast<__nv_fp8_storage_t>(byte), __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half*>(&h));
}
MOE_DEVINL uint32_t float_to_e4m3(float v) {
  return static_cast<uint32_t>(__nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3));
}
// Block scale exponent for a block whose largest magnitude is amax (> 0): values / 2^s lie in [128, 256)
MOE_DEVINL int block_exp(float amax) { return static_cast<int>((__float_as_uint(amax) >> 23) & 0xFFu) - 127 - 7; }
// v (already divided by the block scale) -> (hi, lo) E4M3 bytes with v = hi + lo / 8
MOE_DEVINL void split_e4m3(float v, uint32_t* hi, uint32_t* lo) {
  const uint32_t h = float_to_e4m3(v);
  *hi = h;
  *lo = float_to_e4m3((v - e4m3_to_float(h)) * 8.0f);
}
MOE_DEVINL float pow2f(int e) { return __uint_as_float(static_cast<uint32_t>(e + 127) << 23); }  // e in [-126, 127]

}  // namespace

template <bool STAGE1>
__global__ void __launch_bounds__(kNatThreads, 1)
ffn_native_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_sc, const NatArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const int K = a.K;
  const NatSmem sm = nat_smem(a.E, K);
  unsigned char* sAct = smem + sm.act;  // [K/128 steps][16 rows][128 bytes], 128-byte swizzle
  unsigned char* sW = smem + sm.w;      // ring of [256 rows][128 bytes]
  unsigned char* sSc = smem + sm.sc;    // ring of [256 rows][16 bytes]
  unsigned char* sSfa = smem + sm.sfa;  // [16 rows][K/32] scale bytes of the activation rows
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  uint64_t* full_w = bars;                       // [kWStages]  TMA -> MMA
  uint64_t* empty_w = full_w + kWStages;         // [kWStages]  MMA done -> producer
  uint64_t* full_sc = empty_w + kWStages;        // [kScStages] TMA -> scale warps
  uint64_t* empty_sc = full_sc + kScStages;      // [kScStages] scale warps -> producer
  uint64_t* sf_full = empty_sc + kScStages;      // [kSfGroups] scale warps -> MMA
  uint64_t* sf_free = sf_full + kSfGroups;       // [kSfGroups] MMA done -> scale warps
  uint64_t* acc_full = sf_free + kSfGroups;      // MMA -> epilogue
  uint64_t* acc_empty = acc_full + 1;            // epilogue -> MMA
  uint64_t* act_ready = acc_empty + 1;           // scale warps -> MMA: activation operand of the current (expert, pass)
  uint64_t* act_free = act_ready + 1;            // MMA done with the activation operand -> scale warps
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sm.misc);
  int* touched = reinterpret_cast<int*>(smem + sm.touched);
  int* s_misc = touched + a.E;

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int n_steps = K / kKStep;
  const int tiles_per_expert = a.R / kTile;

  // ---- setup: touched experts, barriers, tensor memory ----
  if (wid == 2) {
    // lane l looks at experts l, l + 32, ...: all loads are issued before any is used (one memory round trip)
    unsigned has_mask = 0u;
#pragma unroll 8
    for (int i = 0; i < (a.E + 31) / 32; ++i) {
      const int e = i * 32 + lane;
      const int lo = (e < a.E) ? __ldg(a.offsets + e) : 0;
      const int hi = (e < a.E) ? __ldg(a.offsets + e + 1) : 0;
      has_mask |= (hi > lo ? 1u : 0u) << i;
    }
    int run = 0;
    for (int i = 0; i < (a.E + 31) / 32; ++i) {
      const int has = static_cast<int>((has_mask >> i) & 1u);
      int tot;
      const int ex = warp_excl_scan(has, lane, &tot);
      if (has) touched[run + ex] = i * 32 + lane;
      run += tot;
    }
    if (lane == 0) s_misc[0] = run;
  }
  if (tid == 0) {
    for (int s = 0; s < kWStages; ++s) { mbar_init(&full_w[s], 1); mbar_init(&empty_w[s], 1); }
    for (int s = 0; s < kScStages; ++s) { mbar_init(&full_sc[s], 1); mbar_init(&empty_sc[s], 4); }
    for (int s = 0; s < kSfGroups; ++s) { mbar_init(&sf_full[s], 4); mbar_init(&sf_free[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 1);
    mbar_init(act_ready, 4);
    mbar_init(act_free, 1);
    mbar_fence_init();
  }
  if (wid == 1) tmem_alloc(tmem_holder, kNatTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  // Programmatic dependent launch: the next grid (down projection after gate/up, combine after down) may start its
  // set-up - and the down projection its weight stream - while this grid is still running; it waits
  // (griddepcontrol.wait) before it reads what this grid writes.  This grid in turn reads nothing of its own
  // predecessor before its scale warps have waited (below), apart from expert_offsets, which the router finished
  // before that predecessor was allowed to start this grid.
  pdl_launch_dependents();
  const int n_touched = s_misc[0];
  const long long total_items = static_cast<long long>(n_touched) * tiles_per_expert;
  const long long per_cta = (total_items + gridDim.x - 1) / gridDim.x;
  const long long item_begin = static_cast<long long>(blockIdx.x) * per_cta;
  const long long item_end = min(item_begin + per_cta, total_items);
  // Every role walks the same sequence: for each item, for each pass of up to 8 tokens, all K steps.

  if (wid == 0) {
    // =========================== producer ===========================
    if (lane == 0) {
      int s = 0, cs = 0;
      uint32_t ph = 0, cph = 0;
      for (long long it = item_begin; it < item_end; ++it) {
        const int e = touched[it / tiles_per_expert];
        const int tile = static_cast<int>(it % tiles_per_expert);
        const int rows = a.offsets[e + 1] - a.offsets[e];
        const int n_pass = (rows + kMaxTokPass - 1) / kMaxTokPass;
        const int wrow_a = STAGE1 ? e * a.R + tile * 128 : e * a.R + tile * kTile;
        const int wrow_b = STAGE1 ? e * a.R + a.I + tile * 128 : wrow_a + 128;
        for (int pass = 0; pass < n_pass; ++pass) {
          for (int ks = 0; ks < n_steps; ++ks) {
            if ((ks & 3) == 0) {
              mbar_wait(&empty_sc[cs], cph ^ 1u, a.status);
              mbar_expect_tx(&full_sc[cs], kScStage);
              tma_load_2d(sSc + cs * kScStage, &tmap_sc, ks * 4, wrow_a, &full_sc[cs]);
              tma_load_2d(sSc + cs * kScStage + 128 * 16, &tmap_sc, ks * 4, wrow_b, &full_sc[cs]);
              if (++cs == kScStages) { cs = 0; cph ^= 1u; }
            }
            mbar_wait(&empty_w[s], ph ^ 1u, a.status);
            mbar_expect_tx(&full_w[s], kWStage / 2);  // the transaction count is in packed (global) bytes
            tma_load_2d(sW + s * kWStage, &tmap_w, ks * kKStep, wrow_a, &full_w[s]);
            tma_load_2d(sW + s * kWStage + 128 * 128, &tmap_w, ks * kKStep, wrow_b, &full_w[s]);
            if (++s == kWStages) { s = 0; ph ^= 1u; }
          }
        }
      }
    }
  } else if (wid == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      int s = 0, slot = 0;
      uint32_t ph = 0, sph = 0, aph = 0, acc_ph = 0;
      int prev_e = -1;
      const uint32_t act_base = smem_u32(sAct);
      const uint32_t d_addr = tmem_base + kColD;
      for (long long it = item_begin; it < item_end; ++it) {
        const int e = touched[it / tiles_per_expert];
        const int rows = a.offsets[e + 1] - a.offsets[e];
        const int n_pass = (rows + kMaxTokPass - 1) / kMaxTokPass;
        for (int pass = 0; pass < n_pass; ++pass) {
          // The activation operand is shared by consecutive items of an expert whose rows fit one pass;
          // otherwise every (item, pass) has its own.  The scale warps follow the same rule.
          const bool new_operand = (prev_e != e) || (n_pass > 1);
          prev_e = e;
          if (new_operand) {
            mbar_wait(act_ready, aph, a.status);
            aph ^= 1u;
          }
          mbar_wait(acc_empty, acc_ph ^ 1u, a.status);
          tc_fence_after_sync();
          for (int ks = 0; ks < n_steps; ++ks) {
            if ((ks & 3) == 0) mbar_wait(&sf_full[slot], sph, a.status);  // weight scale factors of 4 K steps at a time
            mbar_wait(&full_w[s], ph, a.status);
            tc_fence_after_sync();
            const uint32_t w_addr = smem_u32(sW + s * kWStage);
            const uint32_t sf_act = tmem_base + kColSfAct + static_cast<uint32_t>(ks * 4);
            const uint32_t sf_w = tmem_base + kColSfW + static_cast<uint32_t>(slot * 32 + (ks & 3) * 8);
#pragma unroll
            for (uint32_t j = 0; j < 4; ++j)
              umma_mxf4(d_addr, umma_desc_k_sw128(act_base + ks * 2048 + j * 32), umma_desc_k_sw128(w_addr + j * 32),
                        idesc_mxf4(j), sf_act, sf_w, (ks | static_cast<int>(j)) != 0 ? 1u : 0u);
            umma_commit(&empty_w[s]);
            if (++s == kWStages) { s = 0; ph ^= 1u; }
            if ((ks & 3) == 3) {
              umma_commit(&sf_free[slot]);
              if (++slot == kSfGroups) { slot = 0; sph ^= 1u; }
            }
          }
          umma_commit(acc_full);
          acc_ph ^= 1u;
          bool next_new = true;  // is this the last use of the activation operand?
          if (pass + 1 >= n_pass && it + 1 < item_end) next_new = (touched[(it + 1) / tiles_per_expert] != e) || (n_pass > 1);
          if (next_new) umma_commit(act_free);
        }
      }
    }
  } else if (wid >= 2 && wid < 6) {
    // =========================== scale factors and the activation operand ===========================
    const int qq = wid & 3;                      // tensor-memory lane quadrant written by this warp (warps 2..5 -> 2,3,0,1)
    const uint32_t lane_base = static_cast<uint32_t>(qq * 32) << 16;
    const int st = tid - 64;                     // 0..127
    int cs = 0, slot = 0;
    uint32_t cph = 0, sfree_ph = 0, afree_ph = 0;
    int prev_e = -1;
    bool first_op = true;
    for (long long it = item_begin; it < item_end; ++it) {
      const int e = touched[it / tiles_per_expert];
      const int row_begin = a.offsets[e], row_end = a.offsets[e + 1];
      const int n_pass = (row_end - row_begin + kMaxTokPass - 1) / kMaxTokPass;
      for (int pass = 0; pass < n_pass; ++pass) {
        const bool new_operand = (prev_e != e) || (n_pass > 1);
        prev_e = e;
        if (new_operand) {
          // ---- lay out the activation operand of (expert, pass): 8 token rows -> 16 E4M3 rows + scale bytes ----
          if (!first_op) {
            mbar_wait(act_free, afree_ph, a.status);  // MMAs that read the previous operand are done
            afree_ph ^= 1u;
          }
          first_op = false;
          const int row0 = row_begin + pass * kMaxTokPass;
          const int n_tok = min(kMaxTokPass, row_end - row0);
          const int n_blk = K / 32;
          if (STAGE1) {
            pdl_wait();  // the sorted token rows of moe_permute are complete
            // task = (token j, 32-element block b) over the tokens that exist: operand rows of absent tokens keep
            // whatever shared memory holds - their accumulator lanes are never read and rows do not mix
            for (int task = st; task < n_tok * n_blk; task += 128) {
              const int j = task / n_blk, b = task % n_blk;
              uint32_t hi_w[8], lo_w[8];
              uint32_t sb_hi, sb_lo;
              {
                const uint4* src = reinterpret_cast<const uint4*>(a.x + static_cast<size_t>(row0 + j) * K + b * 32);
                uint4 v[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) v[c] = __ldcg(src + c);
                const uint32_t* w32 = reinterpret_cast<const uint32_t*>(v);
                float f[32];
                float amax = 0.0f;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  f[2 * i] = __uint_as_float(w32[i] << 16);
                  f[2 * i + 1] = __uint_as_float(w32[i] & 0xFFFF0000u);
                  amax = fmaxf(amax, fmaxf(fabsf(f[2 * i]), fabsf(f[2 * i + 1])));
                }
                int se = (amax > 0.0f) ? block_exp(amax) : 0;
                se = max(-120, min(se, 120));
                const float inv = pow2f(-se);
                sb_hi = static_cast<uint32_t>(se + 127);
                sb_lo = static_cast<uint32_t>(se - 3 + 127);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  uint32_t hw = 0u, lw = 0u;
#pragma unroll
                  for (int t = 0; t < 4; ++t) {
                    uint32_t h, l;
                    split_e4m3(f[4 * i + t] * inv, &h, &l);
                    hw |= h << (8 * t);
                    lw |= l << (8 * t);
                  }
                  hi_w[i] = hw;
                  lo_w[i] = lw;
                }
              }
              const int ks = b >> 2, c16 = (b & 3) * 2;  // K step, first 16-byte chunk of the 128-byte row
              unsigned char* base = sAct + ks * 2048;
              const int rh = j, rl = 8 + j;  // operand rows 0..7 = hi, 8..15 = lo of tokens 0..7
              *reinterpret_cast<uint4*>(base + rh * 128 + (((c16) ^ (rh & 7)) << 4)) = make_uint4(hi_w[0], hi_w[1], hi_w[2], hi_w[3]);
              *reinterpret_cast<uint4*>(base + rh * 128 + (((c16 + 1) ^ (rh & 7)) << 4)) = make_uint4(hi_w[4], hi_w[5], hi_w[6], hi_w[7]);
              *reinterpret_cast<uint4*>(base + rl * 128 + (((c16) ^ (rl & 7)) << 4)) = make_uint4(lo_w[0], lo_w[1], lo_w[2], lo_w[3]);
              *reinterpret_cast<uint4*>(base + rl * 128 + (((c16 + 1) ^ (rl & 7)) << 4)) = make_uint4(lo_w[4], lo_w[5], lo_w[6], lo_w[7]);
              sSfa[rh * n_blk + b] = static_cast<unsigned char>(sb_hi);
              sSfa[rl * n_blk + b] = static_cast<unsigned char>(sb_lo);
            }
          } else {
            pdl_wait();  // stage 1 is complete and its writes are visible
            // stage 2: the split rows were written by stage 1; copy 16-byte chunks into the swizzled layout
            // operand row r = 8 * half + j (half 0 = hi, 1 = lo) comes from row 2 * (row0 + j) + half of the split
            // activations; only the rows of tokens that exist are copied, four 16-byte chunks in flight per thread
            const int chunks_per_row = K / 16;
            const int n_chunks = 2 * n_tok * chunks_per_row;
            for (int base = st; base < n_chunks; base += 4 * 128) {
              uint4 v[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                const int task = base + u * 128;
                if (task < n_chunks) {
                  const int jj = task / chunks_per_row, c = task % chunks_per_row;
                  const int half = jj >= n_tok ? 1 : 0, j = jj - half * n_tok;
                  v[u] = __ldcg(reinterpret_cast<const uint4*>(a.aq + (static_cast<size_t>(2 * (row0 + j) + half)) * K + c * 16));
                }
              }
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                const int task = base + u * 128;
                if (task < n_chunks) {
                  const int jj = task / chunks_per_row, c = task % chunks_per_row;
                  const int half = jj >= n_tok ? 1 : 0, r = 8 * half + jj - half * n_tok;
                  const int ks = c >> 3, c16 = c & 7;
                  *reinterpret_cast<uint4*>(sAct + ks * 2048 + r * 128 + ((c16 ^ (r & 7)) << 4)) = v[u];
                }
              }
            }
            for (int task = st; task < 2 * n_tok * n_blk; task += 128) {
              const int jj = task / n_blk, b = task % n_blk;
              const int half = jj >= n_tok ? 1 : 0, j = jj - half * n_tok;
              sSfa[(8 * half + j) * n_blk + b] = a.aq_sf[(static_cast<size_t>(2 * (row0 + j) + half)) * n_blk + b];
            }
          }
          fence_proxy_async_smem();
          asm volatile("bar.sync 3, 128;" ::: "memory");
          __syncwarp();
          // activation scale factors -> tensor memory: the block of K step ks holds, in lane n (< 16) of every
          // quadrant, the 4 scale bytes of operand row n for that step
          for (int ks = 0; ks < n_steps; ++ks) {
            const uint32_t w = (lane < 16) ? *reinterpret_cast<const uint32_t*>(sSfa + lane * n_blk + ks * 4) : 0u;
            tmem_st_32x4(tmem_base + lane_base + kColSfAct + static_cast<uint32_t>(ks * 4), w, 0u, 0u, 0u);
          }
          tmem_st_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(act_ready);
        }
        // ---- weight scale factors: one scale stage (256 rows x 16 bytes = 4 K steps) -> one 32-column group ----
        for (int ks = 0; ks < n_steps; ks += 4) {
          mbar_wait(&full_sc[cs], cph, a.status);
          mbar_wait(&sf_free[slot], sfree_ph ^ 1u, a.status);
          __syncwarp();  // the spins may leave lanes diverged; tcgen05.st is warp-collective
          const unsigned char* blk = sSc + cs * kScStage;
          uint4 r[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) r[c] = *reinterpret_cast<const uint4*>(blk + (lane + 32 * c) * 16);
          // column 8t + c of the group: scale bytes of K step t for weight row lane + 32c
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
              "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(
                  tmem_base + lane_base + kColSfW + static_cast<uint32_t>(slot * 32)),
              "r"(r[0].x), "r"(r[1].x), "r"(r[2].x), "r"(r[3].x), "r"(r[4].x), "r"(r[5].x), "r"(r[6].x), "r"(r[7].x),
              "r"(r[0].y), "r"(r[1].y), "r"(r[2].y), "r"(r[3].y), "r"(r[4].y), "r"(r[5].y), "r"(r[6].y), "r"(r[7].y),
              "r"(r[0].z), "r"(r[1].z), "r"(r[2].z), "r"(r[3].z), "r"(r[4].z), "r"(r[5].z), "r"(r[6].z), "r"(r[7].z),
              "r"(r[0].w), "r"(r[1].w), "r"(r[2].w), "r"(r[3].w), "r"(r[4].w), "r"(r[5].w), "r"(r[6].w), "r"(r[7].w)
              : "memory");
          tmem_st_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(&sf_full[slot]);
            mbar_arrive(&empty_sc[cs]);
          }
          if (++cs == kScStages) { cs = 0; cph ^= 1u; }
          if (++slot == kSfGroups) { slot = 0; sfree_ph ^= 1u; }
        }
      }
    }
  } else if (wid == kEpiWarp) {
    // =========================== epilogue (tensor-memory lanes 0..7 = hi, 8..15 = lo of tokens 0..7) ===========================
    // The 16x256b load hands thread t lane t/4 and lane t/4 + 8 of the same two columns: hi + lo is thread-local.
    uint32_t acc_ph = 0;
    const int j = lane >> 2, cp = lane & 3;  // token of this thread, column pair inside a group of 8 columns
    for (long long it = item_begin; it < item_end; ++it) {
      const int e = touched[it / tiles_per_expert];
      const int tile = static_cast<int>(it % tiles_per_expert);
      const int row_begin = a.offsets[e], row_end = a.offsets[e + 1];
      const int n_pass = (row_end - row_begin + kMaxTokPass - 1) / kMaxTokPass;
      for (int pass = 0; pass < n_pass; ++pass) {
        const int p = row_begin + pass * kMaxTokPass + j;  // sorted row of this thread's token
        mbar_wait(acc_full, acc_ph, a.status);
        __syncwarp();  // tcgen05.ld is warp-collective
        acc_ph ^= 1u;
        tc_fence_after_sync();
        if (STAGE1) {
          const int n_blk = a.I / 32;
#pragma unroll 1
          for (int m = 0; m < 4; ++m) {  // 32 consecutive i: gate in columns 32m.., up in columns 128 + 32m..
            uint32_t g[16], u[16];
            tmem_ld_16x256b_x4(tmem_base + kColD + static_cast<uint32_t>(32 * m), g);
            tmem_ld_16x256b_x4(tmem_base + kColD + static_cast<uint32_t>(128 + 32 * m), u);
            tmem_ld_wait();
            if (m == 3) {
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive(acc_empty);  // last read of this accumulator
            }
            float av[8];
            float amax = 0.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
#pragma unroll
              for (int t = 0; t < 2; ++t) {
                const float gv = __uint_as_float(g[4 * i + t]) + __uint_as_float(g[4 * i + 2 + t]);  // hi + lo
                const float uv = __uint_as_float(u[4 * i + t]) + __uint_as_float(u[4 * i + 2 + t]);
                const float sv = __fdividef(gv, 1.0f + __expf(-gv)) * uv;
                av[2 * i + t] = __bfloat162float(__float2bfloat16_rn(sv));  // the intermediate is defined as a bf16 value
                amax = fmaxf(amax, fabsf(av[2 * i + t]));
              }
            }
            // the 32 values of this token's scale block sit in the 4 threads of the token
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            int se = (amax > 0.0f) ? block_exp(amax) : 0;
            se = max(-120, min(se, 120));
            const float inv = pow2f(-se);
            if (p < row_end) {
              const int i0 = tile * 128 + 32 * m;
              uint8_t* dh = a.aq_out + static_cast<size_t>(2 * p) * a.I + i0 + 2 * cp;
              uint8_t* dl = a.aq_out + static_cast<size_t>(2 * p + 1) * a.I + i0 + 2 * cp;
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                uint32_t h0, l0, h1, l1;
                split_e4m3(av[2 * i] * inv, &h0, &l0);
                split_e4m3(av[2 * i + 1] * inv, &h1, &l1);
                *reinterpret_cast<uint16_t*>(dh + 8 * i) = static_cast<uint16_t>(h0 | (h1 << 8));
                *reinterpret_cast<uint16_t*>(dl + 8 * i) = static_cast<uint16_t>(l0 | (l1 << 8));
              }
              if (cp == 0) {
                a.aq_sf_out[static_cast<size_t>(2 * p) * n_blk + (i0 >> 5)] = static_cast<uint8_t>(se + 127);
                a.aq_sf_out[static_cast<size_t>(2 * p + 1) * n_blk + (i0 >> 5)] = static_cast<uint8_t>(se - 3 + 127);
              }
            }
          }
        } else {
#pragma unroll 1
          for (int m = 0; m < 4; ++m) {  // 64 consecutive output columns
            uint32_t v[32];
            tmem_ld_16x256b_x8(tmem_base + kColD + static_cast<uint32_t>(64 * m), v);
            tmem_ld_wait();
            if (m == 3) {
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive(acc_empty);
            }
            if (p < row_end) {
              float* dst = a.y + static_cast<size_t>(p) * a.R + tile * kTile + 64 * m + 2 * cp;
#pragma unroll
              for (int i = 0; i < 8; ++i)
                *reinterpret_cast<float2*>(dst + 8 * i) =
                    make_float2(__uint_as_float(v[4 * i]) + __uint_as_float(v[4 * i + 2]),
                                __uint_as_float(v[4 * i + 1]) + __uint_as_float(v[4 * i + 3]));
            }
          }
        }
      }
    }
  }

  // ---- teardown ----
  tc_fence_before_sync();
  __syncthreads();
  if (wid == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kNatTmemCols);
  }
}

// ---- host side ---------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn nat_encode_fn() {
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

bool nat_map(CUtensorMap* m, CUtensorMapDataType dt, const void* base, uint64_t inner_elems, uint64_t row_bytes, uint64_t rows,
             uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = nat_encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {inner_elems, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool native_shape_ok(const moe_shape_t& sh, const void* w13, const void* w2) {
  // decode-sized: on average at most 32 rows per expert (4 passes of 8 tokens over the weight stream)
  const long long S = static_cast<long long>(sh.T) * sh.k;
  return S <= 4096 && S <= 32LL * sh.E && sh.H % 128 == 0 && sh.I % 128 == 0 && sh.H <= kMaxK && sh.I <= kMaxK && sh.H % 512 == 0 &&
         sh.I % 512 == 0 && (reinterpret_cast<uintptr_t>(w13) & 31u) == 0 && (reinterpret_cast<uintptr_t>(w2) & 31u) == 0 &&
         nat_smem(sh.E, sh.H > sh.I ? sh.H : sh.I).total + 1024 <= 227 * 1024;
}

size_t native_scratch_bytes(const moe_shape_t& sh) {
  const size_t S = static_cast<size_t>(sh.T) * sh.k;
  return align_up(2 * S * sh.I, kAlign) + align_up(2 * S * (sh.I / 32), kAlign);
}

int launch_expert_ffn_native(const __nv_bfloat16* x_perm, const int* offsets, const uint8_t* w13, const uint8_t* s13,
                             const uint8_t* w2, const uint8_t* s2, const moe_shape_t& sh, void* scratch, float* y_perm,
                             int* status_word, cudaStream_t st) {
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(ffn_native_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(ffn_native_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return MOE_ERR_CUDA;
    attr_done = true;
  }
  const size_t S = static_cast<size_t>(sh.T) * sh.k;
  uint8_t* aq = static_cast<uint8_t*>(scratch);
  uint8_t* aq_sf = aq + align_up(2 * S * sh.I, kAlign);
  CUtensorMap tm_w13, tm_w2, tm_s13, tm_s2;
  if (!nat_map(&tm_w13, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, w13, sh.H, sh.H / 2, static_cast<uint64_t>(sh.E) * 2 * sh.I, kKStep,
               128, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !nat_map(&tm_w2, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, w2, sh.I, sh.I / 2, static_cast<uint64_t>(sh.E) * sh.H, kKStep, 128,
               CU_TENSOR_MAP_SWIZZLE_128B) ||
      !nat_map(&tm_s13, CU_TENSOR_MAP_DATA_TYPE_UINT8, s13, sh.H / 32, sh.H / 32, static_cast<uint64_t>(sh.E) * 2 * sh.I, 16, 128,
               CU_TENSOR_MAP_SWIZZLE_NONE) ||
      !nat_map(&tm_s2, CU_TENSOR_MAP_DATA_TYPE_UINT8, s2, sh.I / 32, sh.I / 32, static_cast<uint64_t>(sh.E) * sh.H, 16, 128,
               CU_TENSOR_MAP_SWIZZLE_NONE))
    return MOE_ERR_CUDA;
  const int grid = sm_count();
  NatArgs a;
  a.x = x_perm;
  a.aq = aq;
  a.aq_sf = aq_sf;
  a.aq_out = aq;
  a.aq_sf_out = aq_sf;
  a.offsets = offsets;
  a.y = y_perm;
  a.status = status_word;
  a.E = sh.E;
  a.I = sh.I;
  a.K = sh.H;
  a.R = 2 * sh.I;
  if (launch_pdl(ffn_native_kernel<true>, dim3(grid), dim3(kNatThreads), nat_smem(sh.E, sh.H).total + 1024, st, tm_w13, tm_s13,
                 a) != cudaSuccess)
    return MOE_ERR_CUDA;
  a.K = sh.I;
  a.R = sh.H;
  if (launch_pdl(ffn_native_kernel<false>, dim3(grid), dim3(kNatThreads), nat_smem(sh.E, sh.I).total + 1024, st, tm_w2, tm_s2,
                 a) != cudaSuccess)
    return MOE_ERR_CUDA;
  note_kernel("ffn_native_mxf4_block_scaled", 2);
  return MOE_OK;
}

}  // namespace moe
