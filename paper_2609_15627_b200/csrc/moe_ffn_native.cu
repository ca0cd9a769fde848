// Expert FFN for decode-sized batches on the native block-scaled FP4 tensor-core path:
// packed E2M1 codes and E8M0 scales go HBM -> TMA -> shared memory -> tcgen05.mma with no ALU expansion and
// no padding (shared memory holds the weights exactly as HBM does).
//
// tcgen05.mma kind::mxf4.block_scale multiplies two E2M1 operands with one UE8M0 scale per 32 K elements on
// both sides - the checkpoint format of the expert weights is exactly such an operand - at twice the rate of
// the 8-bit kinds (M = 128, N = 256, K = 64 in 128 cycles: 64 bytes of packed weights per cycle and SM).
// The activations are bf16, so each row is written as a sum of kTerms = 8 E2M1 rows with their own block scales,
//   x = sum_t 2^(s_t) * q_t,   q_t = e2m1(r_t / 2^(s_t)),   r_0 = x,   r_(t+1) = r_t - 2^(s_t) * q_t   (exact),
// with s_t the smallest exponent for which the block's largest |r_t| is at most 6 * 2^(s_t).  Every term removes
// at least two bits of the block's largest residual, so after 8 terms the residual of every element is below
// 2^-16 of its block's largest magnitude, and elements within 2^-10 of it are exact; products are exact and
// accumulate in fp32 in tensor memory.  The 8 rows of a token are 8 of the 128 rows of the A operand, which the
// tensor core walks anyway: the terms cost shared memory, not time.
//
// Operand roles: the weights are the B operand (N = 256 weight rows per MMA, K = 64) and the tokens the A
// operand (M = 128 rows = up to 16 tokens x 8 terms per pass over the weights, row = 8 * token + term; rows of
// tokens that do not exist hold other rows' data or zeros and their accumulator lanes are never looked at).
// Both operands ride the same shared-memory ring: a stage is one K step (256 elements) of the weight tile plus
// the same K step of the pass's term rows, each fetched by TMA with the 128-byte swizzle the MMA reads.
//
// Launches per call: native_split_kernel (token rows -> E2M1 terms, once per row; clears the per-expert completion
// counters), then ffn_native_kernel, in which one persistent CTA per SM runs both projections back to back:
// phase 0 = gate/up + SwiGLU (work item = touched expert x 128 gate rows + the 128 matching up rows, so gate and up of
// one i are two columns of the same accumulator lane), phase 1 = down (item = touched expert x 256 rows).  The weight
// stream runs on across the phase change; a down item loads its term rows once the gate/up items of its expert - its
// own and other CTAs' - have published theirs (one counter per expert, release/acquire through L2, bounded wait).
// No gate/up item ever waits for another CTA, and a down item waits only for gate/up items of CTAs with a lower or
// equal index (see cta_shares), so the waits cannot form a cycle and do not need the whole grid to be resident.
// Warp roles:
//   warp 0      producer: TMA loads of the weight tile, of the term rows and of the weight scale bytes
//   warp 1      allocates tensor memory, issues the MMAs, commits to mbarriers
//   warps 2..5  move weight scale bytes into tensor memory (tcgen05.st), and at a change of (expert, pass) the
//               scale bytes of its term rows
//   warps 6..9  epilogue, one warp per tensor-memory lane quadrant: sum the 8 term rows of each token, then SwiGLU +
//               bf16 rounding + the 8-term split for the down projection (gate/up) or the fp32 store (down).  A pass
//               of more than 4 tokens: quadrant q holds tokens 4q..4q+3, its warp takes all 256 columns.  A pass of
//               at most 4 tokens is loaded into every quadrant, and each warp takes a quarter of the columns.
// Every wait is bounded and reports through the status word.
//
// The weights are read either in the checkpoint's row layout or in moe_prepack's tile-contiguous layout (one tensor
// map box = one contiguous run; see ExpertWeights), always with the L2 evict-first policy: each byte is used once.
//
// Reductions that are multiples of 256 but not of 512 (the I = 256 shard): the scale bytes' rows are then not multiples
// of 16 bytes, which no tensor map addresses; the scale warps fetch them with plain loads instead (Phase::direct).
//
// The same kernel, instantiated with kFused = true, is the whole layer in one launch for a handful of tokens
// (where the one-token kernel does not take the shape): it routes, sorts the slots and splits the token rows itself, and
// reduces over the slots at the end (see FusedArgs).
//
// Instantiated with kQ = true it is the quantised-activation variant (moe_expert_ffn_q): one operand row per token - the
// activation quantised online to E2M1 with one scale per 32 elements, as the paper's historical decode route does to
// INT8 - so a pass holds 128 tokens and the epilogues sum nothing across lanes.  Large batches run one projection per
// launch over blocks of (expert, pass, four tiles) dealt round-robin to the CTAs (see the set-up).
#include <cuda.h>
#include <cuda_fp4.h>

#include <algorithm>
#include <cstring>

#include "moe_mxf4_device.cuh"
#include "moe_tmap.cuh"
#include "moe_route_device.cuh"
#include "moe_sm100_primitives.cuh"

namespace moe {

namespace {

constexpr int kTile = 256;            // weight rows per item (N of the MMA)
constexpr int kKStep = 256;           // K elements per stage: one 128-byte swizzled row of packed codes per weight row
constexpr int kWStage = kTile * 128;  // 32 KB of weights per stage, shared memory and HBM alike
constexpr int kAStage = 128 * 128;    // 16 KB: the same K step of up to 128 term rows
constexpr int kStage = kWStage + kAStage;
constexpr int kWStages = 4;
constexpr int kScStages = 3;          // scale-byte ring: one stage = 256 rows x 16 bytes = 2 K steps
constexpr int kScStage = kTile * 16;
constexpr int kSfGroups = 3;          // tensor-memory groups for the weight scale factors: 4 words x 8 columns
constexpr int kMaxTokPass = 16;       // tokens per pass (16 x 8 = 128 operand rows)
constexpr int kQOneLaunchRows = 64;   // quantised-activation variant: up to this many rows per expert on average, one launch
constexpr int kMaxK = 4096;           // scale factors of one pass's term rows stay in tensor memory: 8 columns per K step
constexpr int kNatThreads = 10 * 32;
constexpr int kEpiWarp = 6;           // warps 6..9: warp % 4 = 2, 3, 0, 1 -> one tensor-memory lane quadrant each
constexpr uint32_t kNatTmemCols = 512;
// tensor-memory columns: one 256-column accumulator; per K step two scale words per operand row, each its own
// scale-factor block of 4 columns (a block covers 128 rows - rows 32c..32c+31 in column c - and must start on a
// multiple of 4 columns); 3 groups of 4 words x 8 columns (256 weight rows) for the weight scales
constexpr uint32_t kColD = 0, kColSfAct = 256, kColSfW = 384;

struct NatArgs {
  const uint8_t* sf1;        // scale bytes of the token rows' terms [S * 8, H/32] (terms: row p * 8 + t, packed E2M1)
  uint8_t* aq2;              // terms of the bf16 intermediate [S * 8, I/2]: written by phase 0, read by phase 1
  uint8_t* sf2;              //   and their scale bytes [S * 8, I/32]
  int* done;                 // [E] epilogue warps that have published a gate/up item of the expert
  const int* offsets;
  float* y;                  // output [S, H]
  float* const* row_dst;     // or null; else output row p goes to row_dst[p] (see y_row)
  int* status;               // never null: the caller's word or the library's own (see StatusRef)
  int own_status;            // the library's own word: the one-launch kernel's last CTA clears it for the next call
  int E, H, I, S;
  int blocked;               // weights in moe_prepack's tile-contiguous layout (see ExpertWeights)
  const uint8_t* s13;        // the weights' scale bytes in the row layout, for reductions that are not multiples of 512:
  const uint8_t* s2;         //   their rows are then not multiples of 16 bytes, which a tensor map cannot address
  int ph_lo, ph_hi;          // projections this launch runs: [0, 2) = both; the large-batch schedule runs one per launch
  int by_pass;               // large-batch schedule: the list of experts is a list of (expert, pass) entries (see the set-up)
};

// The one-launch layer (moe_forward on a handful of tokens): what the kernel needs beyond the expert FFN's arguments.
// Every CTA routes all T tokens itself (same arithmetic, same result everywhere) and sorts the T * k slots by expert in
// shared memory, so its weight stream starts without waiting for anyone.  The first kSplitCtas CTAs meanwhile split
// the T token rows into E2M1 term rows (stored by token: no sorted copy of the rows exists), a few 32-element blocks
// each, and count themselves in; every CTA sees that count complete before its set-up ends (CTAs are handed out in
// index order, so those CTAs are running).  A gate/up item fetches the term rows of its expert's tokens one token (8
// rows) at a time, through the sorted-row -> token table of the slot sort.  After the down projection the CTA that runs the last expert's item of a column tile
// reduces that tile over the slots of every token.
// Tokens the one-launch kernel can take: one routing warp each.  moe_forward uses it for ONE token only: measured at the
// production shape on prepacked weights, 32.7 us against 35.0 us for the four calls at 1 token, but 52.6 against 50.5
// at 2, 85 against 69 at 3, 108 against 85 at 4 - with several items per CTA the set-up that cannot overlap anything
// (routing before the first weight address is known) and the extra hand-over before the final reduction outweigh the
// launches saved.  moe_debug_forward_one_launch runs it for 2 to 4 tokens, for the tests.
constexpr int kFusedMaxTok = 4;
constexpr int kFusedPreferredTok = 1;
constexpr int kFusedMaxSlots = 32; // T * k: one warp sorts them
// The CTAs that split the token rows wait for one another (every other wait in the kernel points to CTAs with a lower
// index), so the grid needs this many SMs to itself at the start; 16 CTAs x 20 groups of 8 lanes cover the 256 blocks of
// two 4096-wide rows in one round, more CTAs would not make it shorter.
constexpr int kSplitCtas = 16;
struct FusedArgs {
  const float* logits;       // [T, E]
  const __nv_bfloat16* x;    // [T, H]
  __nv_bfloat16* out;        // [T, H]
  int* ids_out;              // [T, k] or null
  float* w_out;              // [T, k] or null
  uint8_t* aq1;              // [T * 8, H/2] term rows of the tokens
  uint8_t* sf1;              // [T * 8, H/32]
  int* sync;                 // sync block: [0, E) = NatArgs::done, then the indices above; zero between calls
  int T, k;
};

// Term-row tensor maps of one projection's input: the same tensor with boxes of 8, 16, 32, 64 and 128 rows (1, 2, 4, 8,
// 16 tokens); a pass fetches the smallest box that holds its tokens - every byte of term rows competes with the weights
// for the path from L2
constexpr int kTermBoxes = 5;
struct alignas(64) TermMaps {
  CUtensorMap box[kTermBoxes];
};
// A pass of one token is loaded once per lane quadrant of the accumulator, so that each of the four epilogue warps finds
// the token in its own quadrant and takes a quarter of the columns instead of one warp taking them all (decode_c1:
// every expert has one row, and the epilogues are on the critical path).  The scheme works for up to 4 tokens (one
// quadrant = 32 operand rows), but every repeated KB of term rows competes with the weight stream: measured on
// decode_c64 (2.3 rows per expert on average) the expert-FFN call takes 545 us with passes of up to 4 tokens repeated,
// 526 us with single-token passes only (row-layout weights; 560 against 550 us under the power cap).
// Nor is it worth anything where the epilogue hides behind the next item's MMAs: a CTA repeats only in a phase in which
// it has at most kRepMaxItems items (another 0.7 % on decode_c64, where a CTA has 24).
constexpr int kRepBox = 0, kRepTok = 1 << kRepBox;  // boxes 0..kRepBox hold at most kRepTok tokens
constexpr int kRepMaxItems = 2;
MOE_DEVINL int op_box(int n_rows) { return n_rows <= 8 ? 0 : (n_rows <= 16 ? 1 : (n_rows <= 32 ? 2 : (n_rows <= 64 ? 3 : 4))); }

// One projection as the kernel sees it
struct Phase {
  int K, R, n_steps, tiles;  // reduction length, weight rows per expert, K steps, items per entry of the expert list
  int begin, end;            // this CTA's items (at most 1024 experts x 32 tiles)
  bool direct;               // K is not a multiple of 512: scale bytes come by plain loads (see NatArgs::s13)
  bool rep_ok;               // few enough of them for single-token passes to be repeated per lane quadrant
};
// Items go to CTAs in contiguous shares: gate/up items evenly, per0 each.  A down item of expert t is placed as if it
// followed that expert's last gate/up item in the gate/up list, its expert's down items spread over the span of the
// next expert's gate/up items: with t = i1 / tiles1 and j = i1 % tiles1,
//   u(i1) = (t + 1) * tiles0 - 1 + ceil((j + 1) * tiles0 / tiles1),   CTA(i1) = min(grid - 1, u(i1) / per0).
// So a down item only ever waits for gate/up items of CTAs with a lower or equal index: CTAs are handed out in index
// order, hence whatever a running CTA waits for has been started before it, whether or not the whole grid is
// resident at once.  The shares stay within one expert's items of even.
//
// The smallest down item (of total1) that reaches CTA c, i.e. with u(i1) >= c * per0
__host__ __device__ inline int first_down_item_of_cta(int c, int total1, int tiles0, int tiles1, int per0) {
  const int U = c * per0;
  int t = (U + tiles0) / tiles0 - 2;
  if (t < 0) t = 0;
  const int V = U - (t + 1) * tiles0 + 1;  // need ceil((j + 1) * tiles0 / tiles1) >= V
  int j = V <= 1 ? 0 : ((V - 1) * tiles1) / tiles0;
  if (j >= tiles1) {
    t += 1;
    j = 0;
  }
  const int i1 = t * tiles1 + j;
  return i1 < total1 ? i1 : total1;
}
// CTA c's share of either phase (item counts fit 32 bits: at most 1024 experts x 32 tiles): begin0, end0, begin1, end1
__host__ __device__ inline void cta_shares(int grid, int c, int n_touched, int tiles0, int tiles1, int* out) {
  const int total0 = n_touched * tiles0, total1 = n_touched * tiles1;
  const int per0 = (total0 + grid - 1) / grid;
  out[0] = c * per0 < total0 ? c * per0 : total0;
  out[1] = out[0] + per0 < total0 ? out[0] + per0 : total0;
  out[2] = total1 == 0 ? 0 : first_down_item_of_cta(c, total1, tiles0, tiles1, per0);
  out[3] = total1 == 0 ? 0 : (c + 1 >= grid ? total1 : first_down_item_of_cta(c + 1, total1, tiles0, tiles1, per0));
}
// Large-batch schedule: consecutive tiles of one (expert, pass) entry that a CTA takes in one go
__host__ __device__ inline int block_tiles(int tiles) { return tiles % 4 == 0 ? 4 : (tiles % 2 == 0 ? 2 : 1); }
MOE_DEVINL Phase phase_of(int ph, const NatArgs& a, const int* shares) {
  Phase p;
  p.K = ph == 0 ? a.H : a.I;
  p.R = ph == 0 ? 2 * a.I : a.H;
  p.n_steps = p.K / kKStep;
  p.direct = (p.K % 512) != 0;
  p.tiles = a.by_pass ? block_tiles(p.R / kTile) : p.R / kTile;
  p.begin = shares[2 * ph];
  p.end = shares[2 * ph + 1];
  p.rep_ok = p.end - p.begin <= kRepMaxItems;
  return p;
}

// entries of the list of experts with rows that a CTA keeps
__host__ __device__ inline int touched_cap(int E) { return E > 32 ? E : 32; }
struct NatSmem {
  uint32_t act, w, sc, sfa, bars, misc, touched, route, total;
};
__host__ __device__ inline NatSmem nat_smem(int E, int K) {
  NatSmem m;
  uint32_t off = 0;
  m.act = off;
  m.w = off;  // ring of [256 weight rows][128 bytes] + [128 term rows][128 bytes]
  off += kWStages * kStage;
  m.sc = off;
  off += kScStages * kScStage;
  m.sfa = off;  // [128 term rows][K/32 scale bytes] of the current pass
  off += 128 * (static_cast<uint32_t>(K) / 32);
  m.bars = off;
  off += 64 * 8;
  m.misc = off;
  off += 64;
  m.touched = off;  // touched experts: id, first row, end row
  off += (4 * static_cast<uint32_t>(touched_cap(E)) + 8) * 4;
  m.route = off;    // one-launch layer: expert and weight of every slot, sorted row of every slot, row of (touched expert, token)
  off += 4 * kFusedMaxSlots * 4;
  m.total = off;
  return m;
}

}  // namespace

// ---- split kernel: bf16 token rows -> 8 E2M1 term rows with their scale bytes; 8 threads per 32-element block ----
// Few, large CTAs: the FFN grid's CTAs need a whole SM each and are handed out in blockIdx order, so every SM this
// grid still occupies delays one of them - with at most (SMs - working FFN CTAs) CTAs here, only idle ones.
__global__ void __launch_bounds__(1024) native_split_kernel(const __nv_bfloat16* __restrict__ x, uint8_t* __restrict__ aq,
                                                           uint8_t* __restrict__ aq_sf, int* __restrict__ done, int S, int H,
                                                           int E, int* __restrict__ status_clear) {
  pdl_launch_dependents();  // the FFN grid may set up and start its weight stream; it waits before it reads aq or done
  pdl_wait();               // the sorted token rows of moe_permute are complete, and every earlier kernel on the stream
  const int n_blk = H / 32;
  const long long gt = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gt < E) done[gt] = 0;
  // the library's own status word (caller passed none): whatever an earlier call left there is over, and the FFN grid
  // of this call looks at the word only in waits that have lasted a millisecond
  if (gt == 0 && status_clear != nullptr) *status_clear = 0;
  const long long task = gt >> 3;  // (row, block); the grid is padded to whole warps, so whole tasks are in or out
  const int sub = static_cast<int>(gt & 7);
  const bool live = task < static_cast<long long>(S) * n_blk;
  const int p = live ? static_cast<int>(task / n_blk) : 0, b = live ? static_cast<int>(task % n_blk) : 0;
  const uint2 v = __ldcg(reinterpret_cast<const uint2*>(x + static_cast<size_t>(p) * H + b * 32 + sub * 4));
  float r[1][4] = {{__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                   __uint_as_float(v.y & 0xFFFF0000u)}};
  split_terms<1>(r, [&](int, int t, uint32_t bytes, int se) {
    if (live) {
      const size_t row = static_cast<size_t>(p) * kTerms + t;
      *reinterpret_cast<uint16_t*>(aq + row * (H / 2) + b * 16 + sub * 2) = static_cast<uint16_t>(bytes);
      if (sub == 0) aq_sf[row * n_blk + b] = static_cast<uint8_t>(se + 127);
    }
  });
}

// ---- the quantised-activation variant's split: bf16 token rows -> one E2M1 row with its scale bytes.  Four threads per
// 32-element block, eight consecutive values each (16-byte loads, 4-byte stores: a warp writes 128 contiguous bytes) ----
__global__ void __launch_bounds__(1024) native_quant_rows_kernel(const __nv_bfloat16* __restrict__ x, uint8_t* __restrict__ aq,
                                                                uint8_t* __restrict__ aq_sf, int* __restrict__ done, int S, int H,
                                                                int E, int* __restrict__ status_clear) {
  pdl_launch_dependents();  // as native_split_kernel
  pdl_wait();
  const long long gt = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gt < E) done[gt] = 0;
  if (gt == 0 && status_clear != nullptr) *status_clear = 0;
  const long long n_grp = static_cast<long long>(S) * (H / 8);  // a multiple of 4: whole blocks are in or out
  const bool live = gt < n_grp;
  const uint4 v = live ? __ldcg(reinterpret_cast<const uint4*>(x) + gt) : make_uint4(0u, 0u, 0u, 0u);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  float f[8];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    f[2 * j] = __uint_as_float(w[j] << 16);
    f[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
  float amax = 0.0f;
#pragma unroll
  for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fabsf(f[j]));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
  const int se = (amax > 0.0f) ? term_exp(amax) : 0;
  const float inv = pow2f(-se);
  uint32_t codes = 0u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float qa, qb;
    codes |= e2m1_pair(f[2 * j] * inv, f[2 * j + 1] * inv, &qa, &qb) << (8 * j);
  }
  if (live) {
    reinterpret_cast<uint32_t*>(aq)[gt] = codes;                 // row p, bytes 4 * (group in the row): the same index
    if ((gt & 3) == 0) aq_sf[gt >> 2] = static_cast<uint8_t>(se + 127);  // [row][block]: the same index again
  }
}

// kFused = false: the expert FFN (moe_expert_ffn).  kFused = true: the whole layer in this one launch (see FusedArgs);
// the differences are the set-up, where the gate/up items' operand rows come from, which rows their epilogue writes,
// and the reduction over slots after the down items.
// kQ = true: the quantised-activation variant of the expert FFN.  Every operand row is one token's single E2M1 term
// (the first term of the split: smallest block scale without saturation, round to nearest even), so a pass holds up to
// 128 tokens, nothing is summed over lanes, and the gate/up epilogue quantises the bf16 intermediate the same way.
template <bool kFused, bool kQ = false>
__global__ void __launch_bounds__(kNatThreads, 1)
ffn_native_kernel(const __grid_constant__ CUtensorMap tmap_w13, const __grid_constant__ CUtensorMap tmap_s13,
                  const __grid_constant__ TermMaps tmap_a1, const __grid_constant__ CUtensorMap tmap_w2,
                  const __grid_constant__ CUtensorMap tmap_s2, const __grid_constant__ TermMaps tmap_a2, const NatArgs a,
                  const FusedArgs f) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const NatSmem sm = nat_smem(a.E, a.H > a.I ? a.H : a.I);
  unsigned char* sW = smem + sm.w;      // ring of stages: [256 weight rows][128 bytes] then [128 term rows][128 bytes]
  unsigned char* sSc = smem + sm.sc;    // ring of [256 rows][16 bytes]
  unsigned char* sSfa = smem + sm.sfa;  // [128 term rows][K/32] scale bytes of the current pass
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  uint64_t* full_w = bars;                       // [kWStages]  TMA -> MMA
  uint64_t* empty_w = full_w + kWStages;         // [kWStages]  MMA done -> producer
  uint64_t* full_sc = empty_w + kWStages;        // [kScStages] TMA -> scale warps
  uint64_t* empty_sc = full_sc + kScStages;      // [kScStages] scale warps -> producer
  uint64_t* sf_full = empty_sc + kScStages;      // [kSfGroups] scale warps -> MMA
  uint64_t* sf_free = sf_full + kSfGroups;       // [kSfGroups] MMA done -> scale warps
  uint64_t* acc_full = sf_free + kSfGroups;      // MMA -> epilogue
  uint64_t* acc_empty = acc_full + 1;            // epilogue -> MMA
  uint64_t* act_ready = acc_empty + 1;           // scale warps -> MMA: term-row scale factors of the current (expert, pass)
  uint64_t* act_free = act_ready + 1;            // MMA done with them -> scale warps
  uint64_t* ctr_done = act_free + 1;             // one-launch layer: epilogue warps that are through with the global counters
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sm.misc);
  int* touched = reinterpret_cast<int*>(smem + sm.touched);  // ids of the experts that have rows
  int* t_begin = touched + touched_cap(a.E);                 // their first sorted row
  int* t_end = t_begin + touched_cap(a.E);                   // and the row after their last
  int* t_tile = t_end + touched_cap(a.E);                    // first tile of the entry's items (0 outside the large-batch schedule)
  int* s_misc = t_tile + touched_cap(a.E);
  int* s_ids = reinterpret_cast<int*>(smem + sm.route);                 // [T * k] expert of every slot (one-launch layer only)
  float* s_w = reinterpret_cast<float*>(s_ids + kFusedMaxSlots);        // [T * k] routing weight
  int* s_row = reinterpret_cast<int*>(s_w + kFusedMaxSlots);            // [T * k] sorted row of every slot
  int* s_tok = s_row + kFusedMaxSlots;                                  // [T * k] token of every sorted row

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  static_assert(!(kFused && kQ), "the one-launch layer has no quantised-activation variant");
  constexpr int nt = kQ ? 1 : kTerms;                 // operand rows per token
  constexpr int tok_pass = kQ ? 128 : kMaxTokPass;    // tokens per pass: 128 operand rows
  const int need_done = 4 * (2 * a.I / kTile);  // four epilogue warps publish each gate/up item of an expert

  // ---- setup: touched experts, barriers, tensor memory ----
  if (tid == 32 * 3) {  // a warp with nothing to set up fetches the tensor maps
    prefetch_tmap(&tmap_w13);
    prefetch_tmap(&tmap_s13);
    prefetch_tmap(&tmap_w2);
    prefetch_tmap(&tmap_s2);
    for (int i = 0; i < kTermBoxes; ++i) {
      prefetch_tmap(&tmap_a1.box[i]);
      prefetch_tmap(&tmap_a2.box[i]);
    }
  }
  if (!kFused && a.by_pass && wid == 2) {
    // Large-batch schedule (one projection per launch, so no item waits for another).  The list of experts becomes a
    // list of (expert, pass) entries of at most tok_pass rows, each cut into blocks of a few consecutive tiles
    // (block_tiles); block b goes to CTA b mod gridDim.x.  So every item is one pass and equal block counts are equal
    // work (an expert with many rows would otherwise make its items many passes long); the items of a block share the
    // operand's scale factors in tensor memory; and at any moment the grid works on neighbouring blocks - a few experts'
    // weights and token rows, which stay in L2 for the other passes and tiles that need them (with one contiguous share
    // per CTA every pass re-read its expert's weights from DRAM: 7 GB instead of 2.3 in the gate/up launch at
    // prefill_8k).  A CTA keeps one list entry per block of its own: slot j = block blockIdx.x + j * gridDim.x.
    const int tiles = a.ph_lo == 0 ? 2 * a.I / kTile : a.H / kTile;
    const int bt = block_tiles(tiles), bpe = tiles / bt;  // tiles per block, blocks per entry
    const int grid = static_cast<int>(gridDim.x), c = static_cast<int>(blockIdx.x);
    const int n_it = (a.E + 31) / 32;
    int run = 0;
    for (int i = 0; i < n_it; ++i) {
      const int e = i * 32 + lane;
      const int lo = (e < a.E) ? __ldg(a.offsets + e) : 0;
      const int hi = (e < a.E) ? __ldg(a.offsets + e + 1) : 0;
      const int v = (hi - lo + tok_pass - 1) / tok_pass;
      int tot;
      const int first = run + warp_excl_scan(v, lane, &tot);
      // blocks [first * bpe, (first + v) * bpe) belong to this expert; mine are those = c (mod grid)
      const long long b_lo = static_cast<long long>(first) * bpe, b_hi = static_cast<long long>(first + v) * bpe;
      long long b = b_lo <= c ? c : c + (b_lo - c + grid - 1) / grid * grid;
      for (; b < b_hi; b += grid) {
        const int slot = static_cast<int>((b - c) / grid), vi = static_cast<int>(b / bpe) - first;
        if (slot < touched_cap(a.E)) {  // (the host chooses this schedule only where the list fits)
          touched[slot] = e;
          t_tile[slot] = static_cast<int>(b % bpe) * bt;
          t_begin[slot] = lo + vi * tok_pass;
          t_end[slot] = min(hi, lo + (vi + 1) * tok_pass);
        }
      }
      run += tot;
    }
    if (lane == 0) {
      const long long n_blocks = static_cast<long long>(run) * bpe;
      const int n_slots = n_blocks > c ? static_cast<int>((n_blocks - c + grid - 1) / grid) : 0;
      s_misc[0] = n_slots;
      s_misc[1] = s_misc[2] = s_misc[3] = s_misc[4] = 0;
      s_misc[2 + 2 * a.ph_lo] = min(n_slots, touched_cap(a.E)) * bt;
    }
  } else if (!kFused && wid == 2) {
    // lane l looks at experts l, l + 32, ...: all loads are issued before any is used (one memory round trip);
    // the second loop's loads hit L1.  expert_offsets was complete before the permute kernel let this chain start.
    const int n_it = (a.E + 31) / 32;
    unsigned has_mask = 0u;
#pragma unroll 8
    for (int i = 0; i < n_it; ++i) {
      const int e = i * 32 + lane;
      const int lo = (e < a.E) ? __ldg(a.offsets + e) : 0;
      const int hi = (e < a.E) ? __ldg(a.offsets + e + 1) : 0;
      has_mask |= (hi > lo ? 1u : 0u) << i;
    }
    int run = 0;
    for (int i = 0; i < n_it; ++i) {
      const int has = static_cast<int>((has_mask >> i) & 1u);
      int tot;
      const int ex = warp_excl_scan(has, lane, &tot);
      if (has) {
        const int e = i * 32 + lane;
        touched[run + ex] = e;
        t_tile[run + ex] = 0;
        t_begin[run + ex] = __ldg(a.offsets + e);
        t_end[run + ex] = __ldg(a.offsets + e + 1);
      }
      run += tot;
    }
    if (lane == 0) {
      s_misc[0] = run;
      cta_shares(static_cast<int>(gridDim.x), static_cast<int>(blockIdx.x), run, 2 * a.I / kTile, a.H / kTile, s_misc + 1);
    }
  }
  if (tid == 0) {
    for (int s = 0; s < kWStages; ++s) { mbar_init(&full_w[s], 1); mbar_init(&empty_w[s], 1); }
    for (int s = 0; s < kScStages; ++s) { mbar_init(&full_sc[s], 1); mbar_init(&empty_sc[s], 4); }
    for (int s = 0; s < kSfGroups; ++s) { mbar_init(&sf_full[s], 4); mbar_init(&sf_free[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 4);
    mbar_init(act_ready, 4);
    mbar_init(act_free, 1);
    mbar_init(ctr_done, 4);
    mbar_fence_init();
  }
  // Operand rows that no term-row box has written yet read as zeros instead of whatever shared memory held (their
  // results are never looked at; zeros cost less power)
  for (int s = 0; s < kWStages; ++s) {
    uint4* z = reinterpret_cast<uint4*>(sW + s * kStage + kWStage);
    for (int i = tid; i < kAStage / 16; i += kNatThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  fence_proxy_async_smem();
  if (wid == 1) tmem_alloc(tmem_holder, kNatTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  // Programmatic dependent launch: the next grid on the stream (moe_combine) may start its set-up now; it waits
  // (griddepcontrol.wait) for this grid to complete before it reads the output.  This grid in turn reads nothing
  // of the split kernel before it has waited itself, apart from expert_offsets (see above).
  pdl_launch_dependents();
  if constexpr (kFused) {
    // ---- the layer's first steps, the same in every CTA: route, sort the slots, split the token rows ----
    pdl_wait();  // logits and token rows may come from the kernel before this one; the sync block is clear
    const int n_split = min(static_cast<int>(gridDim.x), kSplitCtas);
    if (tid == 0) {
      const int dirty = __ldcg(f.sync + kSyncCanary0) | __ldcg(f.sync + kSyncCanary1);
      s_misc[5] = dirty;
      if (dirty != 0 && a.status != nullptr) atomicExch(a.status, static_cast<int>(MOE_ERR_WORKSPACE));
    }
    // the thread that adds to and polls the split count looks for itself (it runs before the CTA's first barrier)
    int dirty32 = 0;
    if (tid == 32) dirty32 = __ldcg(f.sync + kSyncCanary0) | __ldcg(f.sync + kSyncCanary1);
    if (wid >= 2 && wid < 6) {
      // one warp per token: top-k by logit (ties to the lower expert), softmax over the selected logits
      const int t = wid - 2;
      if (t < f.T) {
        float* row = reinterpret_cast<float*>(sSfa) + t * a.E;  // this region is not in use yet
        for (int e0 = 0; e0 < a.E; e0 += 256) {  // eight loads in flight per lane
          float lv[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int e = e0 + 32 * u + lane;
            lv[u] = e < a.E ? __ldg(f.logits + static_cast<size_t>(t) * a.E + e) : 0.0f;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int e = e0 + 32 * u + lane;
            if (e < a.E) row[e] = lv[u];
          }
        }
        __syncwarp();
        int my_id;
        float my_v;
        warp_topk(row, a.E, f.k, lane, &my_id, &my_v);
        const float wt = warp_softmax_selected(my_v, f.k, lane);
        if (lane < f.k) {
          s_ids[t * f.k + lane] = my_id;
          s_w[t * f.k + lane] = wt;
          if (blockIdx.x == 0 && f.ids_out != nullptr) f.ids_out[t * f.k + lane] = my_id;
          if (blockIdx.x == 0 && f.w_out != nullptr) f.w_out[t * f.k + lane] = wt;
        }
      }
    } else if (wid != 0 && static_cast<int>(blockIdx.x) < n_split) {
      // warps 1 and 6..9 of the first CTAs: token rows -> term rows, one 32-element block per group of 8 lanes;
      // CTA c takes blocks c, c + n_split, ..., 20 of them per round (one round up to two 4096-wide rows)
      const int sw = wid == 1 ? 0 : wid - 5;  // 0..4
      const int n_blk = a.H / 32, n_all = f.T * n_blk;
      const int sub = lane & 7;
      const int n_rounds = (n_all + n_split * 20 - 1) / (n_split * 20);
      for (int rd = 0; rd < n_rounds; ++rd) {
        const int b = static_cast<int>(blockIdx.x) + n_split * (rd * 20 + sw * 4 + (lane >> 3));
        const bool live = b < n_all;
        const int t = live ? b / n_blk : 0, blk = live ? b % n_blk : 0;
        const uint2 v = *reinterpret_cast<const uint2*>(f.x + static_cast<size_t>(t) * a.H + blk * 32 + sub * 4);
        float r[1][4] = {{__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                         __uint_as_float(v.y & 0xFFFF0000u)}};
        split_terms<1>(r, [&](int, int t8, uint32_t bytes, int se) {
          if (live) {
            const size_t trow = static_cast<size_t>(t) * kTerms + t8;
            *reinterpret_cast<uint16_t*>(f.aq1 + trow * (a.H / 2) + blk * 16 + sub * 2) = static_cast<uint16_t>(bytes);
            if (sub == 0) f.sf1[trow * n_blk + blk] = static_cast<uint8_t>(se + 127);
          }
        });
      }
      fence_proxy_async_all();  // TMA will read these rows
      asm volatile("bar.sync 2, 160;" ::: "memory");  // the five splitting warps
      if (tid == 32 && dirty32 == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(f.sync + kSyncSplit) : "memory");
    }
    __syncthreads();
    // the term rows are complete by the time the routing above is: one thread makes sure while the slots are sorted
    if (tid == 32 && dirty32 == 0) counter_wait_ge(f.sync + kSyncSplit, n_split, a.status);
    if (wid == 2) {
      // Stable sort of the slots by expert, S <= 32: lane s is slot s.  Its sorted row = slots of smaller experts +
      // earlier slots of its own expert; the touched experts are the distinct ids in ascending order.
      const int S = f.T * f.k;
      const int id = lane < S ? s_ids[lane] : 0x7fffffff;
      int less = 0, eq_all = 0, eq_before = 0;
      for (int o = 0; o < S; ++o) {
        const int oid = __shfl_sync(0xffffffffu, id, o);
        less += oid < id;
        eq_all += oid == id;
        eq_before += (oid == id) && (o < lane);
      }
      const bool first = lane < S && eq_before == 0;
      int ti = 0;  // touched experts with a smaller id
      for (int o = 0; o < S; ++o) {
        const int oid = __shfl_sync(0xffffffffu, id, o);
        const int of = __shfl_sync(0xffffffffu, static_cast<int>(first), o);
        ti += of && (oid < id);
      }
      const int n_t = __popc(__ballot_sync(0xffffffffu, first));
      if (lane < S) {
        s_row[lane] = less + eq_before;
        s_tok[less + eq_before] = lane / f.k;
      }
      if (first) {
        touched[ti] = id;
        t_tile[ti] = 0;
        t_begin[ti] = less;
        t_end[ti] = less + eq_all;
      }
      if (lane == 0) {
        s_misc[0] = n_t;
        cta_shares(static_cast<int>(gridDim.x), static_cast<int>(blockIdx.x), n_t, 2 * a.I / kTile, a.H / kTile, s_misc + 1);
      }
    }
    __syncthreads();
  }
  // Every role walks the same sequence: both phases; in each, this CTA's items; per item, passes of up to tok_pass
  // tokens; per pass, all K steps.

  const int role = (kFused && s_misc[5] != 0) ? -1 : wid;  // a sync block that was never cleared: no work at all
  if (role == 0) {
    // =========================== producer ===========================
    if (lane == 0) {
      int s = 0, cs = 0;
      uint32_t ph = 0, cph = 0;
      // every weight byte is read once per call - unless items have several passes, each of which reads it again
      const uint64_t stream_once = a.by_pass ? l2_policy_evict_normal() : l2_policy_evict_first();
      // The weights depend on nothing, the term rows do: on the split kernel (phase 0) or on the gate/up items of
      // their expert (phase 1).  While a dependency is open, the weight loads go out and the term-row loads of up to
      // kWStages steps are held back; they follow once the dependency is met.
      // (one-launch layer: the tokens' term rows were seen complete during the set-up)
      bool pdl_done = kFused, dep_ok = kFused;
      if (kFused) fence_proxy_async_all();  // they were written through the generic proxy
      int dep_phase = 0, dep_e = -1;
      int n_pend = 0, pend_s[kWStages], pend_x[kWStages], pend_y[kWStages], pend_b[kWStages], pend_r[kWStages];
      // term rows of one K step, n_rep times: once, or once per lane quadrant of the accumulator
      auto load_terms = [&](const TermMaps* ma, int stage, int bi, int n_rep, int x, int y) {
        for (int r = 0; r < n_rep; ++r)
          tma_load_2d(sW + stage * kStage + kWStage + r * (32 * 128), &ma->box[bi], x, y, &full_w[stage]);
      };
      auto meet = [&]() {  // wait for the open dependency and send the held-back loads
        if (!pdl_done) {
          pdl_wait();  // the split kernel is complete: term rows of the tokens, cleared counters
          pdl_done = true;
        }
        if (dep_phase == 1) {
          counter_wait_ge(a.done + dep_e, need_done, a.status);
          fence_proxy_async_all();  // the rows were written through the generic proxy, TMA reads through the async one
        }
        const TermMaps* ma = dep_phase == 0 ? &tmap_a1 : &tmap_a2;
        for (int i = 0; i < n_pend; ++i) load_terms(ma, pend_s[i], pend_b[i], pend_r[i], pend_x[i], pend_y[i]);
        n_pend = 0;
        dep_ok = true;
      };
      for (int phase = a.ph_lo; phase < a.ph_hi; ++phase) {
        const Phase P = phase_of(phase, a, s_misc + 1);
        const CUtensorMap* mw = phase == 0 ? &tmap_w13 : &tmap_w2;
        const CUtensorMap* msc = phase == 0 ? &tmap_s13 : &tmap_s2;
        const TermMaps* ma = phase == 0 ? &tmap_a1 : &tmap_a2;
        for (int it = P.begin; it < P.end; ++it) {
          const int ti = it / P.tiles, e = touched[ti];
          const int tile = t_tile[ti] + it % P.tiles;
          const int row_begin = t_begin[ti];
          const int n_rows_e = t_end[ti] - row_begin;
          const int n_pass = (n_rows_e + tok_pass - 1) / tok_pass;
          const int wrow_a = phase == 0 ? e * P.R + tile * 128 : e * P.R + tile * kTile;
          const int wrow_b = phase == 0 ? e * P.R + a.I + tile * 128 : wrow_a + 128;
          if (phase == 1 && (dep_phase != 1 || dep_e != e)) {  // a new dependency: settle the old one first
            if (n_pend > 0) meet();
            dep_phase = 1;
            dep_e = e;
            dep_ok = false;
          }
          for (int pass = 0; pass < n_pass; ++pass) {
            const bool by_token = kFused && phase == 0;  // the expert's rows are fetched token by token (at most 4)
            const int bi = op_box(min(tok_pass, n_rows_e - pass * tok_pass) * nt);  // box of 8 << bi operand rows
            const int n_rep = (!kQ && P.rep_ok && bi <= kRepBox) ? 4 : 1;
            for (int ks = 0; ks < P.n_steps; ++ks) {
              if (!P.direct && (ks & 1) == 0) {  // 16 scale bytes per weight row cover two K steps
                mbar_wait(&empty_sc[cs], cph ^ 1u, a.status);
                mbar_expect_tx(&full_sc[cs], kScStage);
                // 128 rows x 16 scale bytes; tile-contiguous layout: tile (row / 128, ks / 2) is 128 consecutive rows of 16 bytes
                const int sx = a.blocked ? 0 : ks * 8;
                const int sya = a.blocked ? ((wrow_a >> 7) * (P.n_steps >> 1) + (ks >> 1)) * 128 : wrow_a;
                const int syb = a.blocked ? ((wrow_b >> 7) * (P.n_steps >> 1) + (ks >> 1)) * 128 : wrow_b;
                tma_load_2d_hint(sSc + cs * kScStage, msc, sx, sya, &full_sc[cs], stream_once);
                tma_load_2d_hint(sSc + cs * kScStage + 128 * 16, msc, sx, syb, &full_sc[cs], stream_once);
                if (++cs == kScStages) { cs = 0; cph ^= 1u; }
              }
              mbar_wait(&empty_w[s], ph ^ 1u, a.status);
              mbar_expect_tx(&full_w[s], static_cast<uint32_t>(kWStage + n_rep * (by_token ? n_rows_e * 8 : 8 << bi) * 128));
              // 128 rows x 128 bytes of codes; tile-contiguous layout: tile (row / 128, ks) is 128 consecutive rows of 128 bytes
              const int wx = a.blocked ? 0 : ks * 128;
              const int wya = a.blocked ? ((wrow_a >> 7) * P.n_steps + ks) * 128 : wrow_a;
              const int wyb = a.blocked ? ((wrow_b >> 7) * P.n_steps + ks) * 128 : wrow_b;
              tma_load_2d_hint(sW + s * kStage, mw, wx, wya, &full_w[s], stream_once);
              tma_load_2d_hint(sW + s * kStage + 128 * 128, mw, wx, wyb, &full_w[s], stream_once);
              // the pass's term rows (8 per token, consecutive); rows past the end of the tensor arrive as zeros
              const int arow = (row_begin + pass * tok_pass) * nt;
              if (by_token) {
                // (the tokens' term rows were seen complete during the set-up: no dependency to hold these back for)
                for (int j = 0; j < n_rows_e; ++j)
                  for (int r = 0; r < n_rep; ++r)
                    tma_load_2d(sW + s * kStage + kWStage + r * (32 * 128) + j * (8 * 128), &ma->box[0], ks * 128,
                                s_tok[row_begin + j] * kTerms, &full_w[s]);
              } else if (dep_ok) {
                load_terms(ma, s, bi, n_rep, ks * 128, arow);
              } else {
                pend_r[n_pend] = n_rep;
                pend_s[n_pend] = s;
                pend_x[n_pend] = ks * 128;
                pend_y[n_pend] = arow;
                pend_b[n_pend] = bi;
                if (++n_pend == kWStages) meet();
              }
              if (++s == kWStages) { s = 0; ph ^= 1u; }
            }
          }
        }
      }
      if (n_pend > 0) meet();
    }
    if constexpr (kFused) {
      // Once this CTA's last addition to and last read of the counters are behind it (the epilogue warps say so;
      // every other warp's reads come before the MMAs those warps have waited for), it counts itself out, and the last
      // CTA to do so clears the sync block for the next call.  This runs beside the final reduction, not after it.
      int last = 0;
      if (lane == 0) {
        mbar_wait(ctr_done, 0u, a.status);
        __threadfence();
        last = atomicAdd(f.sync + kSyncExit, 1) == static_cast<int>(gridDim.x) - 1;
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        __threadfence();
        for (int i = lane; i < a.E; i += 32) f.sync[i] = 0;
        for (int i = lane; i < a.H / kTile; i += 32) f.sync[kSyncDone2 + i] = 0;
        if (lane == 0) {
          f.sync[kSyncExit] = 0;
          f.sync[kSyncSplit] = 0;
          if (a.own_status) *a.status = 0;  // every wait of this call is over; nobody reads this word on the host
        }
      }
    }
  } else if (role == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      int s = 0, slot = 0;
      uint32_t ph = 0, sph = 0, aph = 0, acc_ph = 0;
      const uint32_t d_addr = tmem_base + kColD;
      for (int phase = a.ph_lo; phase < a.ph_hi; ++phase) {
        const Phase P = phase_of(phase, a, s_misc + 1);
        int prev_ti = -1;
        for (int it = P.begin; it < P.end; ++it) {
          const int ti = it / P.tiles;
          const int n_pass = (t_end[ti] - t_begin[ti] + tok_pass - 1) / tok_pass;
          for (int pass = 0; pass < n_pass; ++pass) {
            // The scale factors of the term rows (tensor memory) are shared by consecutive items of an expert whose
            // rows fit one pass; otherwise every (item, pass) has its own.  The scale warps follow the same rule.
            const bool new_operand = (prev_ti != ti) || (n_pass > 1);
            prev_ti = ti;
            if (new_operand) {
              mbar_wait(act_ready, aph, a.status);
              aph ^= 1u;
            }
            mbar_wait(acc_empty, acc_ph ^ 1u, a.status);
            tc_fence_after_sync();
            for (int ks = 0; ks < P.n_steps; ++ks) {
              if ((ks & 1) == 0) mbar_wait(&sf_full[slot], sph, a.status);  // weight scale factors of 2 K steps at a time
              mbar_wait(&full_w[s], ph, a.status);
              tc_fence_after_sync();
              const uint32_t w_addr = smem_u32(sW + s * kStage);
#pragma unroll
              for (uint32_t j = 0; j < 4; ++j) {  // K = 64 each; scale word (ks & 1) * 2 + j / 2 of the group, half j & 1
                const uint32_t sf_act = tmem_base + kColSfAct + static_cast<uint32_t>(ks * 8) + (j >> 1) * 4;
                const uint32_t sf_w = tmem_base + kColSfW + static_cast<uint32_t>(slot * 32 + ((ks & 1) * 2 + (j >> 1)) * 8);
                umma_mxf4(d_addr, umma_desc_k_sw128(w_addr + kWStage + j * 32), umma_desc_k_sw128(w_addr + j * 32),
                          idesc_mxf4(j & 1u), sf_act, sf_w, (ks | static_cast<int>(j)) != 0 ? 1u : 0u);
              }
              umma_commit(&empty_w[s]);
              if (++s == kWStages) { s = 0; ph ^= 1u; }
              if ((ks & 1) == 1 || ks == P.n_steps - 1) {
                umma_commit(&sf_free[slot]);
                if (++slot == kSfGroups) { slot = 0; sph ^= 1u; }
              }
            }
            umma_commit(acc_full);
            acc_ph ^= 1u;
            // last use of these scale factors?  (always at the end of a phase)
            bool next_new = true;
            if (pass + 1 >= n_pass && it + 1 < P.end) next_new = ((it + 1) / P.tiles != ti) || (n_pass > 1);
            if (next_new) umma_commit(act_free);
          }
        }
      }
    }
  } else if (role >= 2 && role < 6) {
    // =========================== scale factors of the weights and of the term rows ===========================
    const int qq = wid & 3;                      // tensor-memory lane quadrant written by this warp (warps 2..5 -> 2,3,0,1)
    const uint32_t lane_base = static_cast<uint32_t>(qq * 32) << 16;
    const int st = tid - 64;                     // 0..127
    int cs = 0, slot = 0;
    uint32_t cph = 0, sfree_ph = 0, afree_ph = 0;
    bool first_op = true;
    for (int phase = a.ph_lo; phase < a.ph_hi; ++phase) {
      const Phase P = phase_of(phase, a, s_misc + 1);
      const int n_blk = P.K / 32;
      const uint8_t* src_sf = phase == 0 ? (kFused ? f.sf1 : a.sf1) : a.sf2;
      int prev_ti = -1;
      for (int it = P.begin; it < P.end; ++it) {
        const int ti = it / P.tiles;
        const int row_begin = t_begin[ti], row_end = t_end[ti];
        const int n_pass = (row_end - row_begin + tok_pass - 1) / tok_pass;
        for (int pass = 0; pass < n_pass; ++pass) {
          const bool new_operand = (prev_ti != ti) || (n_pass > 1);
          prev_ti = ti;
          if (new_operand) {
            // ---- scale factors of the pass's term rows: global -> shared memory -> tensor memory ----
            if (first_op) {
              if (!kFused) pdl_wait();  // the split kernel is complete: scale bytes of the tokens' terms, cleared counters
            } else {
              mbar_wait(act_free, afree_ph, a.status);  // MMAs that read the previous scale factors are done
              afree_ph ^= 1u;
            }
            first_op = false;
            if (phase == 1) {
              // every gate/up item of this expert has published its rows of the intermediate
              if (st == 0) counter_wait_ge(a.done + touched[ti], need_done, a.status);
              asm volatile("bar.sync 3, 128;" ::: "memory");
            }
            const bool by_token = kFused && phase == 0;  // the tokens' scale bytes are stored by token, not by sorted row
            const int row0 = row_begin + pass * tok_pass;
            const int n_rows = min(tok_pass, row_end - row0) * nt;  // operand rows that exist
            const bool rep = !kQ && P.rep_ok && n_rows <= kRepTok * kTerms;  // the operand repeats in every lane quadrant
            // rows are n_blk bytes each and consecutive: one contiguous range, copied 16 bytes at a time
            // (the 16-byte chunks of a row are XOR-swizzled with the row number against bank conflicts)
            const int n_chunk = n_blk / 16, cmask = min(n_chunk, 8) - 1;
            const int n_vec = n_rows * n_chunk;
            const uint4* src = reinterpret_cast<const uint4*>(src_sf + static_cast<size_t>(row0) * nt * n_blk);
            if (P.direct) {  // rows of n_blk = 8 (mod 16) bytes: 8 bytes at a time, rows plainly one after the other
              const uint2* src8 = reinterpret_cast<const uint2*>(src_sf + static_cast<size_t>(row0) * nt * n_blk);
              for (int i = st; i < n_rows * (n_blk / 8); i += 128) reinterpret_cast<uint2*>(sSfa)[i] = __ldcg(src8 + i);
            } else
            for (int i = st; i < n_vec; i += 128) {
              const int r = i / n_chunk, c = i % n_chunk;
              const uint4* from = by_token ? reinterpret_cast<const uint4*>(src_sf) + (s_tok[row0 + (r >> 3)] * kTerms + (r & 7)) * n_chunk + c
                                           : src + i;
              reinterpret_cast<uint4*>(sSfa)[r * n_chunk + (c ^ (r & cmask))] = __ldcg(from);
            }
            asm volatile("bar.sync 3, 128;" ::: "memory");
            __syncwarp();
            // K step ks owns two scale-factor blocks (its two scale words); column c of a block holds, in lane l of
            // every quadrant, the word of term row 32c + l (rows that do not exist: any value)
            for (int ks = 0; ks < P.n_steps; ++ks) {
              uint32_t w[8];
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const int r = rep ? lane : 32 * c + lane;
                const uint2 v = P.direct ? reinterpret_cast<const uint2*>(sSfa)[r * (n_blk / 8) + ks]
                                         : *reinterpret_cast<const uint2*>(sSfa + (r * n_chunk + ((ks >> 1) ^ (r & cmask))) * 16 + (ks & 1) * 8);
                w[c] = v.x;
                w[4 + c] = v.y;
              }
              tmem_st_32x8(tmem_base + lane_base + kColSfAct + static_cast<uint32_t>(ks * 8), w);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            asm volatile("bar.sync 3, 128;" ::: "memory");  // sSfa may be overwritten only after every warp has read it
            if (lane == 0) mbar_arrive(act_ready);
          }
          // ---- weight scale factors: one scale stage (256 rows x 16 bytes = 2 K steps) -> one 32-column group ----
          for (int ks = 0; ks < P.n_steps; ks += 2) {
            uint4 r[8];
            if (P.direct) {
              // 8 scale bytes per weight row and K step, straight from the row layout; issued before the wait below
              const int e = touched[ti], tile = t_tile[ti] + it % P.tiles;
              const int wrow_a = phase == 0 ? e * P.R + tile * 128 : e * P.R + tile * kTile;
              const int wrow_b = phase == 0 ? e * P.R + a.I + tile * 128 : wrow_a + 128;
              const uint8_t* sc = phase == 0 ? a.s13 : a.s2;
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                const uint2* p = reinterpret_cast<const uint2*>(sc + static_cast<size_t>((c < 4 ? wrow_a : wrow_b) + lane + 32 * (c & 3)) * n_blk) + ks;
                const uint2 lo = __ldg(p);
                const uint2 hi = ks + 1 < P.n_steps ? __ldg(p + 1) : make_uint2(0u, 0u);
                r[c] = make_uint4(lo.x, lo.y, hi.x, hi.y);
              }
            } else {
              mbar_wait(&full_sc[cs], cph, a.status);
            }
            mbar_wait(&sf_free[slot], sfree_ph ^ 1u, a.status);
            __syncwarp();  // the spins may leave lanes diverged; tcgen05.st is warp-collective
            const unsigned char* blk = sSc + cs * kScStage;
            if (!P.direct) {
#pragma unroll
              for (int c = 0; c < 8; ++c) r[c] = *reinterpret_cast<const uint4*>(blk + (lane + 32 * c) * 16);
            }
            // column 8t + c of the group: scale word t (K blocks 4t..4t+3 of the 16) for weight row lane + 32c
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
              if (!P.direct) mbar_arrive(&empty_sc[cs]);
            }
            if (!P.direct && ++cs == kScStages) { cs = 0; cph ^= 1u; }
            if (++slot == kSfGroups) { slot = 0; sfree_ph ^= 1u; }
          }
        }
      }
    }
  } else if (role >= kEpiWarp) {
    // =========================== epilogue ===========================
    // Accumulator lane = term row = 8 * token + term.  A 32x32b load hands each lane 32 columns of its row; three
    // exchange rounds over the 8 lanes of a token (each halves the columns a lane keeps) leave lane (token, t) with
    // the 8-term sums of 4 consecutive columns, at offset 16 (t & 1) + 8 (t >> 1 & 1) + 4 (t >> 2) of the 32.
    // A pass of more than kRepTok tokens: the warp of quadrant q owns tokens 4q..4q+3 and all 256 columns.  A smaller
    // pass has all its tokens in every quadrant: the warp of quadrant q owns a quarter of the columns of every token.
    const int q = wid & 3;
    const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
    const int jl = lane >> 3, tl = lane & 7;
    const int cb = 16 * (tl & 1) + 8 * ((tl >> 1) & 1) + 4 * (tl >> 2);
    uint32_t acc_ph = 0;
    bool told = false;  // one-launch layer: this warp has said that it is through with the global counters
    auto tell = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(ctr_done);
      told = true;
    };
    // One pass of one item.  `dry` runs the same instructions on whatever tensor memory holds, with every wait, signal
    // and store left out: each CTA executes this code only a few times, so its first real use would otherwise pay
    // for fetching it - on the critical path of a one-item CTA - while the warp has nothing to do before the first
    // accumulator is complete.
    auto run_pass = [&](const int phase, const bool rep_ok, const int out_stride, const int tile, const int row0, const int n_tok,
                        const bool dry) {
      const bool rep = rep_ok && n_tok <= kRepTok;
      const bool active = rep || 4 * q < n_tok;
      // 32-column chunks this warp sums: all 8, or (small pass) gate chunk q and up chunk 4 + q of a gate/up item,
      // chunks 2q and 2q + 1 of a down item
      const int n_ch = rep ? 2 : 8;
      const int ch0 = rep ? (phase == 0 ? q : 2 * q) : 0, ch_step = rep ? (phase == 0 ? 4 : 1) : 1;
      if (!dry) {
        mbar_wait(acc_full, acc_ph, a.status);
        acc_ph ^= 1u;
      }
      __syncwarp();  // tcgen05.ld is warp-collective
      tc_fence_after_sync();
      float acc[8][4];  // [chunk][column cb + c of the chunk]
      if (active) {
#pragma unroll
        for (int mm = 0; mm < 8; ++mm) {
          if (mm < n_ch) {
            uint32_t vc[32];
            tmem_ld_32x32(tmem_base + lane_base + kColD + static_cast<uint32_t>(32 * (ch0 + mm * ch_step)), vc);
            tmem_ld_wait();
            float a16[16], a8[8];
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              const float lo = __uint_as_float(vc[k]), hi = __uint_as_float(vc[16 + k]);
              a16[k] = ((tl & 1) ? hi : lo) + __shfl_xor_sync(0xffffffffu, (tl & 1) ? lo : hi, 1);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k)
              a8[k] = ((tl & 2) ? a16[8 + k] : a16[k]) + __shfl_xor_sync(0xffffffffu, (tl & 2) ? a16[k] : a16[8 + k], 2);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              acc[mm][k] = ((tl & 4) ? a8[4 + k] : a8[k]) + __shfl_xor_sync(0xffffffffu, (tl & 4) ? a8[k] : a8[4 + k], 4);
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (!dry && lane == 0) mbar_arrive(acc_empty);  // the accumulator is free: the rest overlaps the next item's MMAs
      if (!active) return;
      if (phase == 0) {
        // SwiGLU, bf16 rounding and the 8-term split, one (token, block of 32 consecutive i) per group of 8 lanes
        const int n_blk_i = a.I / 32;
        // small pass: lane group jl has token jl, block q of the item's four, gate in acc[0] and up in acc[1] - one
        // round.  Otherwise round rd hands the four blocks of the quadrant's token rd (gate in chunk m, up in chunk
        // m + 4) to the four lane groups.
        const int n_rd = rep ? 1 : min(4, n_tok - 4 * q);
#pragma unroll 1
        for (int rd = 0; rd < n_rd; ++rd) {
          float gsel[4], usel[4];
          if (rep) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              gsel[c] = acc[0][c];
              usel[c] = acc[1][c];
            }
          } else {
#pragma unroll
            for (int m = 0; m < 4; ++m)
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const float tg = __shfl_sync(0xffffffffu, acc[m][c], rd * 8 + tl);
                const float tu = __shfl_sync(0xffffffffu, acc[m + 4][c], rd * 8 + tl);
                if (jl == m) {
                  gsel[c] = tg;
                  usel[c] = tu;
                }
              }
          }
          float r[1][4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float sv = __fdividef(gsel[c], 1.0f + __expf(-gsel[c])) * usel[c];
            r[0][c] = __bfloat162float(__float2bfloat16_rn(sv));  // the intermediate is defined as a bf16 value
          }
          const int tok = rep ? jl : 4 * q + rd;  // token of the pass whose block this lane group splits
          const int i0 = tile * 128 + 32 * (rep ? q : jl);
          const bool live = !dry && tok < n_tok;
          uint8_t* qrow = a.aq2 + static_cast<size_t>(row0 + tok) * kTerms * (a.I / 2) + ((i0 + cb) >> 1);
          uint8_t* srow = a.sf2 + static_cast<size_t>(row0 + tok) * kTerms * n_blk_i + (i0 >> 5);
          split_terms<1>(r, [&](int, int t, uint32_t bytes, int se) {
            if (live) {
              *reinterpret_cast<uint16_t*>(qrow + static_cast<size_t>(t) * (a.I / 2)) = static_cast<uint16_t>(bytes);
              if (tl == 0) srow[static_cast<size_t>(t) * n_blk_i] = static_cast<uint8_t>(se + 127);
            }
          });
        }
      } else {
        const int tok = rep ? jl : 4 * q + jl;
        if (!dry && tok < n_tok) {
          float* dst = y_row(a.y, a.row_dst, static_cast<size_t>(row0 + tok), out_stride) + tile * kTile + 32 * ch0 + cb;
#pragma unroll
          for (int mm = 0; mm < 8; ++mm)
            if (mm < n_ch) *reinterpret_cast<float4*>(dst + 32 * mm) = make_float4(acc[mm][0], acc[mm][1], acc[mm][2], acc[mm][3]);
        }
      }
    };
    // Quantised-activation variant: accumulator lane = operand row = token.  The warp of quadrant q owns tokens
    // 32q..32q+31 of the pass and all 256 columns of theirs; nothing is summed across lanes.
    auto run_pass_q = [&](const int phase, const int out_stride, const int tile, const int row0, const int n_tok) {
      const bool active = 32 * q < n_tok;
      const int tok = 32 * q + lane;
      const bool live = tok < n_tok;
      mbar_wait(acc_full, acc_ph, a.status);
      acc_ph ^= 1u;
      __syncwarp();  // tcgen05.ld is warp-collective
      tc_fence_after_sync();
      if (phase == 0) {
        // columns 0..127 gate, 128..255 up of i = tile * 128 + column; SwiGLU and the rounding to bf16 while the
        // accumulator is read (two values per register), its quantisation after the accumulator is handed back
        uint32_t pk[64];
        if (active) {
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            uint32_t g[32], u[32];
            tmem_ld_32x32(tmem_base + lane_base + kColD + static_cast<uint32_t>(32 * b), g);
            tmem_ld_32x32(tmem_base + lane_base + kColD + static_cast<uint32_t>(32 * (4 + b)), u);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float g0 = __uint_as_float(g[2 * j]), g1 = __uint_as_float(g[2 * j + 1]);
              const float v0 = __fdividef(g0, 1.0f + __expf(-g0)) * __uint_as_float(u[2 * j]);
              const float v1 = __fdividef(g1, 1.0f + __expf(-g1)) * __uint_as_float(u[2 * j + 1]);
              const __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);  // the intermediate is defined as a bf16 value
              pk[16 * b + j] = *reinterpret_cast<const uint32_t*>(&h);
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty);  // the rest overlaps the next pass's MMAs
        if (!active) return;
        const int n_blk_i = a.I / 32;
        uint8_t* qrow = a.aq2 + static_cast<size_t>(row0 + tok) * (a.I / 2) + tile * 64;
        uint8_t* srow = a.sf2 + static_cast<size_t>(row0 + tok) * n_blk_i + tile * 4;
#pragma unroll
        for (int b = 0; b < 4; ++b) {  // one block of 32 consecutive i: block scale, then 32 codes = 16 bytes
          float amax = 0.0f;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint32_t w = pk[16 * b + j];
            amax = fmaxf(amax, fmaxf(fabsf(__uint_as_float(w << 16)), fabsf(__uint_as_float(w & 0xFFFF0000u))));
          }
          const int se = (amax > 0.0f) ? term_exp(amax) : 0;
          const float inv = pow2f(-se);
          uint32_t w4[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint32_t w = pk[16 * b + j];
            float qa, qb;
            w4[j >> 2] |= e2m1_pair(__uint_as_float(w << 16) * inv, __uint_as_float(w & 0xFFFF0000u) * inv, &qa, &qb) << (8 * (j & 3));
          }
          if (live) {
            *reinterpret_cast<uint4*>(qrow + 16 * b) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
            srow[b] = static_cast<uint8_t>(se + 127);
          }
        }
      } else {
        if (active) {
          // each lane writes its own row: 32 bytes per store where the output allows it (whole sectors), and the next
          // chunk's tensor-memory load in flight during the stores of the current one
          float* dst = y_row(a.y, a.row_dst, static_cast<size_t>(live ? row0 + tok : row0), out_stride) + tile * kTile;
          const bool wide = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
          auto put = [&](const uint32_t (&v)[32], int m) {
            if (!live) return;
            if (wide) {
#pragma unroll
              for (int j = 0; j < 4; ++j)
                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + 32 * m + 8 * j), "r"(v[8 * j]),
                             "r"(v[8 * j + 1]), "r"(v[8 * j + 2]), "r"(v[8 * j + 3]), "r"(v[8 * j + 4]), "r"(v[8 * j + 5]),
                             "r"(v[8 * j + 6]), "r"(v[8 * j + 7])
                             : "memory");
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(dst + 32 * m + 4 * j) = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            }
          };
          const uint32_t col = tmem_base + lane_base + kColD;
          uint32_t va[32], vb[32];
          tmem_ld_32x32(col, va);
          tmem_ld_wait();
#pragma unroll 1
          for (int m = 0; m < 8; m += 2) {
            tmem_ld_32x32(col + static_cast<uint32_t>(32 * (m + 1)), vb);
            put(va, m);
            tmem_ld_wait();
            if (m + 2 < 8) tmem_ld_32x32(col + static_cast<uint32_t>(32 * (m + 2)), va);
            put(vb, m + 1);
            if (m + 2 < 8) tmem_ld_wait();
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty);
      }
    };
    for (int sweep = kQ ? 1 : 0; sweep < 2; ++sweep) {  // sweep 0 is the dry run of this CTA's first pass, through the one call site below
      const bool dry = sweep == 0;
      for (int phase = dry ? 0 : a.ph_lo; phase < (dry ? 1 : a.ph_hi); ++phase) {
        const Phase P = phase_of(phase, a, s_misc + 1);
        const int it_end = dry ? min(P.begin + 1, P.end) : P.end;
        for (int it = P.begin; it < it_end; ++it) {
          const int ti = it / P.tiles, tile = t_tile[ti] + it % P.tiles;
          const int row_begin = t_begin[ti], row_end = t_end[ti];
          const int n_pass = dry ? 1 : (row_end - row_begin + tok_pass - 1) / tok_pass;
          for (int pass = 0; pass < n_pass; ++pass) {
            const int row0 = row_begin + pass * tok_pass;
            if constexpr (kQ)
              run_pass_q(phase, P.R, tile, row0, min(tok_pass, row_end - row0));
            else
              run_pass(phase, P.rep_ok, P.R, tile, row0, min(tok_pass, row_end - row0), dry);
          }
          if constexpr (kFused) {
            if (!dry && phase == 1) {
              // this warp's columns of the item are stored: count it for the column tile, and after the last
              // expert's item reduce the tile over the slots of every token (in slot order, as moe_combine does)
              __syncwarp();
              if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(f.sync + kSyncDone2 + tile) : "memory");
              if (ti == s_misc[0] - 1) {
                if (lane == 0) counter_wait_ge(f.sync + kSyncDone2 + tile, 4 * s_misc[0], a.status);
                if (it + 1 == P.end) tell();
                __syncwarp();
                const int col = tile * kTile + (wid - kEpiWarp) * 64 + lane * 2;
                for (int t = 0; t < f.T; ++t) {
                  float2 acc = make_float2(0.0f, 0.0f);
                  for (int j0 = 0; j0 < f.k; j0 += 8) {  // eight slots' loads in flight; the multiply-adds stay in slot order
                    float2 v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                      if (j0 + u < f.k)
                        v[u] = __ldcg(reinterpret_cast<const float2*>(a.y + static_cast<size_t>(s_row[t * f.k + j0 + u]) * a.H + col));
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                      if (j0 + u < f.k) {
                        const float wj = s_w[t * f.k + j0 + u];
                        acc.x = __fmaf_rn(wj, v[u].x, acc.x);
                        acc.y = __fmaf_rn(wj, v[u].y, acc.y);
                      }
                  }
                  *reinterpret_cast<__nv_bfloat162*>(f.out + static_cast<size_t>(t) * a.H + col) = __floats2bfloat162_rn(acc.x, acc.y);
                }
              }
            }
          }
          if (!dry && phase == 0) {
            // publish: this warp's rows of the item (all passes) are written; TMA (asynchronous proxy) and plain
            // loads of other CTAs will read them
            fence_proxy_async_all();
            __syncwarp();  // orders the lanes' stores before lane 0's release
            if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.done + touched[ti]) : "memory");
          }
        }
      }
    }
    if (kFused && !told) tell();
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

// byte tensor [rows][row_bytes], box [box_rows][box_bytes]
bool nat_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_bytes, uint32_t box_rows,
             CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = nat_encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {box_bytes, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace {
bool nat_attr_once() {
  static PerDeviceFlag flag;
  return once_per_device(flag, [] {
    return cudaFuncSetAttribute(ffn_native_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess &&
           cudaFuncSetAttribute(ffn_native_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess &&
           cudaFuncSetAttribute(ffn_native_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
  });
}
}  // namespace

// byte tensor [rows][row_bytes] with a 128-byte-swizzled box of [box_rows][128 bytes] (declared in moe_tmap.cuh)
bool term_row_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_rows) {
  return nat_map(m, base, row_bytes, rows, 128, box_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

// bf16 matrix [rows][inner], 128-byte-swizzled box of [box_rows][box_inner]; rows past the end read as zeros
bool bf16_map_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows) {
  EncodeTiledFn fn = nat_encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * 2};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// tensor maps of the weights and their scale bytes, in either layout (declared in moe_tmap.cuh)
bool weight_maps(const ExpertWeights& w, const moe_shape_t& sh, CUtensorMap* tm_w13, CUtensorMap* tm_s13, CUtensorMap* tm_w2,
                 CUtensorMap* tm_s2) {
  const uint64_t r13 = static_cast<uint64_t>(sh.E) * 2 * sh.I, r2 = static_cast<uint64_t>(sh.E) * sh.H;
  if (w.blocked)  // every tile is [128 rows][128 or 16 bytes], tiles one after the other
    return nat_map(tm_w13, w.w13, 128, r13 * (sh.H / 256), 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
           nat_map(tm_w2, w.w2, 128, r2 * (sh.I / 256), 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
           nat_map(tm_s13, w.s13, 16, r13 * (sh.H / 512), 16, 128, CU_TENSOR_MAP_SWIZZLE_NONE) &&
           nat_map(tm_s2, w.s2, 16, r2 * (sh.I / 512), 16, 128, CU_TENSOR_MAP_SWIZZLE_NONE);
  // (scale rows that are not multiples of 16 bytes get no tensor map: the kernel loads them itself)
  std::memset(tm_s13, 0, sizeof(*tm_s13));
  std::memset(tm_s2, 0, sizeof(*tm_s2));
  return nat_map(tm_w13, w.w13, sh.H / 2, r13, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
         nat_map(tm_w2, w.w2, sh.I / 2, r2, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) &&
         (sh.H % 512 != 0 || nat_map(tm_s13, w.s13, sh.H / 32, r13, 16, 128, CU_TENSOR_MAP_SWIZZLE_NONE)) &&
         (sh.I % 512 != 0 || nat_map(tm_s2, w.s2, sh.I / 32, r2, 16, 128, CU_TENSOR_MAP_SWIZZLE_NONE));
}

bool native_q_shape_ok(const moe_shape_t& sh, const void* w13, const void* w2) {
  return sh.H <= kMaxK && sh.I <= kMaxK && sh.H % 256 == 0 && sh.I % 256 == 0 &&
         (reinterpret_cast<uintptr_t>(w13) & 15u) == 0 && (reinterpret_cast<uintptr_t>(w2) & 15u) == 0 &&
         nat_smem(sh.E, sh.H > sh.I ? sh.H : sh.I).total + 1024 <= 227 * 1024;
}

bool native_shape_ok(const moe_shape_t& sh, const void* w13, const void* w2) {
  return native_batch_ok(sh) && sh.H <= kMaxK && sh.I <= kMaxK && sh.H % 256 == 0 && sh.I % 256 == 0 &&
         (reinterpret_cast<uintptr_t>(w13) & 15u) == 0 && (reinterpret_cast<uintptr_t>(w2) & 15u) == 0 &&
         nat_smem(sh.E, sh.H > sh.I ? sh.H : sh.I).total + 1024 <= 227 * 1024;
}

namespace {
// kQ: the quantised-activation variant (one operand row per token instead of kTerms)
template <bool kQ>
int launch_native_ffn(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& sh,
                      void* scratch, float* y_perm, StatusRef status, cudaStream_t st, float* const* row_dst) {
  if (!nat_attr_once()) return MOE_ERR_CUDA;
  const size_t S = static_cast<size_t>(sh.T) * sh.k;
  const size_t rows = S * (kQ ? 1 : kTerms);  // operand rows
  // scratch: operand rows of the intermediate and of the token rows, each followed by its scale bytes; the counters
  uint8_t* aq2 = static_cast<uint8_t*>(scratch);
  uint8_t* sf2 = aq2 + align_up(rows * (sh.I / 2), kAlign);
  uint8_t* aq1 = sf2 + align_up(rows * (sh.I / 32), kAlign);
  uint8_t* sf1 = aq1 + align_up(rows * (sh.H / 2), kAlign);
  int* done = reinterpret_cast<int*>(sf1 + align_up(rows * (sh.H / 32), kAlign));
  CUtensorMap tm_w13, tm_w2, tm_s13, tm_s2;
  TermMaps tm_a1, tm_a2;
  for (int i = 0; i < kTermBoxes; ++i)
    if (!nat_map(&tm_a1.box[i], aq1, sh.H / 2, rows, 128, 8u << i, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !nat_map(&tm_a2.box[i], aq2, sh.I / 2, rows, 128, 8u << i, CU_TENSOR_MAP_SWIZZLE_128B))
      return MOE_ERR_CUDA;
  if (!weight_maps(w, sh, &tm_w13, &tm_s13, &tm_w2, &tm_s2)) return MOE_ERR_CUDA;
  const size_t per_block = kQ ? 4 : 8;  // threads per 32-element block
  const size_t split_threads = S * (sh.H / 32) * per_block > static_cast<size_t>(sh.E) ? S * (sh.H / 32) * per_block : static_cast<size_t>(sh.E);
  const dim3 split_grid(static_cast<unsigned>((split_threads + 1023) / 1024));
  int* own_word = status.own ? status.word : nullptr;
  if ((kQ ? launch_pdl(native_quant_rows_kernel, split_grid, dim3(1024), 0, st, x_perm, aq1, sf1, done, static_cast<int>(S), sh.H, sh.E, own_word)
          : launch_pdl(native_split_kernel, split_grid, dim3(1024), 0, st, x_perm, aq1, sf1, done, static_cast<int>(S), sh.H, sh.E, own_word)) !=
      cudaSuccess)
    return MOE_ERR_CUDA;
  NatArgs a;
  a.sf1 = sf1;
  a.aq2 = aq2;
  a.sf2 = sf2;
  a.done = done;
  a.offsets = offsets;
  a.y = y_perm;
  a.row_dst = row_dst;
  a.status = status.word;
  a.own_status = 0;
  a.E = sh.E;
  a.H = sh.H;
  a.I = sh.I;
  a.S = static_cast<int>(S);
  a.blocked = w.blocked ? 1 : 0;
  a.s13 = w.s13;
  a.s2 = w.s2;
  // Batches whose experts have several passes: one launch per projection, shares balanced by passes (see pass_shares)
  // (a CTA's blocks, one list entry each, must fit the list it keeps)
  const size_t ent_max = S / (kQ ? 128 : kMaxTokPass) + sh.E, grid_n = static_cast<size_t>(sm_count());
  const size_t bpe_max = static_cast<size_t>(std::max(2 * sh.I / kTile / block_tiles(2 * sh.I / kTile), sh.H / kTile / block_tiles(sh.H / kTile)));
  const bool two = kQ && S > static_cast<size_t>(kQOneLaunchRows) * sh.E &&
                   (ent_max * bpe_max + grid_n - 1) / grid_n + 1 <= static_cast<size_t>(touched_cap(sh.E));
  a.by_pass = two ? 1 : 0;
  for (int l = 0; l < (two ? 2 : 1); ++l) {
    a.ph_lo = two ? l : 0;
    a.ph_hi = two ? l + 1 : 2;
    if (launch_pdl(ffn_native_kernel<false, kQ>, dim3(sm_count()), dim3(kNatThreads),
                   nat_smem(sh.E, sh.H > sh.I ? sh.H : sh.I).total + 1024, st, tm_w13, tm_s13, tm_a1, tm_w2, tm_s2, tm_a2, a,
                   FusedArgs{}) != cudaSuccess)
      return MOE_ERR_CUDA;
  }
  note_kernel(kQ ? "ffn_native_mxf4_quantised_activations" : "ffn_native_mxf4_block_scaled", two ? 3 : 2);
  return MOE_OK;
}
}  // namespace

int launch_expert_ffn_native(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& sh,
                             void* scratch, float* y_perm, StatusRef status, cudaStream_t st, float* const* row_dst) {
  return launch_native_ffn<false>(x_perm, offsets, w, sh, scratch, y_perm, status, st, row_dst);
}
int launch_expert_ffn_native_q(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& sh,
                               void* scratch, float* y_perm, StatusRef status, cudaStream_t st, float* const* row_dst) {
  return launch_native_ffn<true>(x_perm, offsets, w, sh, scratch, y_perm, status, st, row_dst);
}

// ---- the one-launch layer ----
// Applies to a handful of tokens on shapes the native variant takes; the router's scratch (T rows of E logits)
// borrows the shared memory that later holds the term rows' scale bytes.
bool forward_fused_ok(const moe_shape_t& sh, const void* w13, const void* w2) {
  const int K = sh.H > sh.I ? sh.H : sh.I;
  return native_shape_ok(sh, w13, w2) && sh.H % 512 == 0 && sh.I % 512 == 0 && sm_count() >= kSplitCtas && sh.T <= kFusedMaxTok && sh.T * sh.k <= kFusedMaxSlots &&
         static_cast<size_t>(sh.T) * sh.E * 4 <= static_cast<size_t>(128) * (K / 32) && sh.E <= kSyncDone2 &&
         sh.H / kTile <= kSyncExit - kSyncDone2;
}
size_t forward_fused_scratch_bytes(const moe_shape_t& sh) {
  const size_t S = static_cast<size_t>(sh.T) * sh.k, own = static_cast<size_t>(sh.T) * kTerms;
  return align_up(S * sh.H * 4, kAlign) + align_up(S * kTerms * (sh.I / 2), kAlign) + align_up(S * kTerms * (sh.I / 32), kAlign) +
         align_up(own * (sh.H / 2), kAlign) + align_up(own * (sh.H / 32), kAlign);
}
bool forward_fused_preferred(const moe_shape_t& sh) { return sh.T <= kFusedPreferredTok; }

int launch_forward_fused(const float* logits, const __nv_bfloat16* x, const ExpertWeights& w, const moe_shape_t& sh,
                         __nv_bfloat16* out, int* ids_out, float* w_out, int* sync, void* scratch, StatusRef status,
                         cudaStream_t st) {
  if (!nat_attr_once()) return MOE_ERR_CUDA;
  const size_t S = static_cast<size_t>(sh.T) * sh.k;
  const int grid = sm_count();
  const size_t own = static_cast<size_t>(sh.T) * kTerms;
  // scratch: per-slot output rows of the down projection, term rows of the intermediate with their scale bytes, and
  // the term rows of the tokens with theirs
  float* y = static_cast<float*>(scratch);
  uint8_t* aq2 = reinterpret_cast<uint8_t*>(y) + align_up(S * sh.H * 4, kAlign);
  uint8_t* sf2 = aq2 + align_up(S * kTerms * (sh.I / 2), kAlign);
  uint8_t* aq1 = sf2 + align_up(S * kTerms * (sh.I / 32), kAlign);
  uint8_t* sf1 = aq1 + align_up(own * (sh.H / 2), kAlign);
  CUtensorMap tm_w13, tm_w2, tm_s13, tm_s2;
  TermMaps tm_a1, tm_a2;
  for (int i = 0; i < kTermBoxes; ++i)
    if (!nat_map(&tm_a1.box[i], aq1, sh.H / 2, own, 128, 8u << i, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !nat_map(&tm_a2.box[i], aq2, sh.I / 2, S * kTerms, 128, 8u << i, CU_TENSOR_MAP_SWIZZLE_128B))
      return MOE_ERR_CUDA;
  if (!weight_maps(w, sh, &tm_w13, &tm_s13, &tm_w2, &tm_s2)) return MOE_ERR_CUDA;
  NatArgs a;
  a.sf1 = nullptr;
  a.aq2 = aq2;
  a.sf2 = sf2;
  a.done = sync;
  a.offsets = nullptr;
  a.y = y;
  a.row_dst = nullptr;
  a.status = status.word;
  a.own_status = status.own ? 1 : 0;
  a.E = sh.E;
  a.H = sh.H;
  a.I = sh.I;
  a.S = static_cast<int>(S);
  a.blocked = w.blocked ? 1 : 0;
  a.s13 = w.s13;
  a.s2 = w.s2;
  a.ph_lo = 0;
  a.ph_hi = 2;
  a.by_pass = 0;
  FusedArgs f;
  f.logits = logits;
  f.x = x;
  f.out = out;
  f.ids_out = ids_out;
  f.w_out = w_out;
  f.aq1 = aq1;
  f.sf1 = sf1;
  f.sync = sync;
  f.T = sh.T;
  f.k = sh.k;
  if (launch_pdl(ffn_native_kernel<true>, dim3(grid), dim3(kNatThreads), nat_smem(sh.E, sh.H > sh.I ? sh.H : sh.I).total + 1024, st,
                 tm_w13, tm_s13, tm_a1, tm_w2, tm_s2, tm_a2, a, f) != cudaSuccess)
    return MOE_ERR_CUDA;
  note_kernel("layer_one_launch_mxf4_block_scaled", 1);
  return MOE_OK;
}

}  // namespace moe

extern "C" int moe_debug_native_cta_share(int32_t n_ctas, int32_t cta, int32_t n_touched, int32_t H, int32_t I, int32_t* out4) {
  if (out4 == nullptr || n_ctas < 1 || cta < 0 || cta >= n_ctas || n_touched < 0 || n_touched > 1024 || H < moe::kTile ||
      I < moe::kTile / 2 || H % moe::kTile != 0 || (2 * I) % moe::kTile != 0)
    return MOE_ERR_INVALID_ARG;
  moe::cta_shares(n_ctas, cta, n_touched, 2 * I / moe::kTile, H / moe::kTile, out4);
  return MOE_OK;
}
