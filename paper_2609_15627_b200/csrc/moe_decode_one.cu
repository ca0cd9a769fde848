// The whole layer for ONE token in one launch (moe_forward at T = 1): route, gate/up + SwiGLU, down, reduction over slots.
//
// A single token leaves every CTA one work item, so nothing is amortised and the step time is a chain of latencies
// around 107 MB of weight streaming.  This kernel is laid out to keep that chain short:
//
//   * No slot sort.  CTA i takes gate/up item i = (slot j = i / tiles, tile = i % tiles) of 128 gate rows + the 128
//     matching up rows.  One warp routes the token (top-k by warp reductions, the fixed-sequence softmax) and hands the
//     expert ids to the TMA-issuing warp, which starts the weight stream at once: the weights depend on nothing else.
//   * The token row is split into its eight E2M1 term rows by the first H/256 CTAs - the earliest to start - 8 blocks of
//     32 elements each, about a microsecond (splitting the whole row in every CTA was tried: several microseconds of
//     issue time).  They store kCopies copies to global memory and count themselves in; every CTA with an item fetches
//     the rows K step by K step with its weight stages (TMA, four copies of each row, one per lane quadrant of the
//     accumulator) and their scale bytes straight into registers on the way to tensor memory.
//   * The down projection is split along K, so that it needs no other CTA's part of the intermediate: the two CTAs of a
//     thread-block cluster hold neighbouring 128-wide slices of the expert's intermediate (gate/up tiles 2p and 2p + 1),
//     exchange their E2M1 term rows through distributed shared memory (st.shared::cluster, one cluster barrier), and
//     each multiplies the joint 256-wide slice - one 128-byte K step of the packed W2 rows, the same tiles and the same
//     tensor maps as everywhere else - with half of the expert's H output rows.  The partial sums go to
//     part[slot][p][H] (fp32, one store per element, no atomics).
//   * The last H/128 CTAs each own 128 output columns: they wait until every partial of their half of the columns is
//     stored (one counter per half, release/acquire), sum the I/256 partials of every slot in ascending p, and combine
//     the k slots in slot order with fma from zero - moe_combine's arithmetic - into the bf16 output row.  Every wait
//     points to CTAs with a lower or equal index.
//   * Code that runs once per launch is fetched cold: the epilogue warps walk their code "dry" (same instructions, no
//     waits, signals or stores) while the first accumulator fills, the reducing CTAs theirs before their count completes.
//     (Dry runs BEFORE griddepcontrol.wait were tried and dropped: a warp whose lane 0 has gone through a loop of its own
//     ran the warp-wide code after it four times slower, and a CTA that starts late pays for the dry run in full.)
//
// The result equals the four calls' up to the summation order inside the down projection's dot products (here I/256
// partial sums added in ascending order, there one accumulator over the whole of I); routing ids and weights are
// bit-identical, the reduction over slots is the defined one.
//
// Warp roles (320 threads, one CTA per SM, clusters of two CTAs):
//   warp 0      lane 0 issues all TMA loads (weights, weight scale bytes, the token's term rows) of both projections
//   warp 1      allocates tensor memory, issues the MMAs (kind::mxf4.block_scale, M = 128 term rows, N = 256 weight rows)
//   warps 2..5  move weight scale bytes shared memory -> tensor memory
//   warps 6..9  epilogue, one per lane quadrant: scale factors of the token's terms -> tensor memory; gate/up
//               accumulator -> SwiGLU -> bf16 -> term rows into both CTAs of the pair; down accumulators -> partial
//               sums.  Warp 8 first routes and waits for the split; warps 6 and 9 of the first CTAs split the token row.
// Every wait on an mbarrier or a counter is bounded and reports through the status word.
#include "moe_mxf4_device.cuh"
#include "moe_route_device.cuh"
#include "moe_tmap.cuh"

namespace moe {

#ifdef MOE_TRACE
__device__ unsigned long long g_one_trace[160][32];
MOE_DEVINL unsigned long long trace_time() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)::"memory");
  return t;
}
#define MOE_TP(i) g_one_trace[blockIdx.x][i] = trace_time()
#else
#define MOE_TP(i)
#endif

namespace {

constexpr int kTile = 256;             // weight rows per MMA (N)
constexpr int kWStage = kTile * 128;   // 32 KB: 256 weight rows x one K step (256 elements = 128 packed bytes)
constexpr int kWStages = 4;
constexpr int kScStage = kTile * 16;   // 4 KB: 256 rows x 16 scale bytes (two K steps)
constexpr int kScStages = 3;
constexpr int kSfGroups = 3;           // tensor-memory groups of weight scale factors: 4 words x 8 columns each
constexpr int kATile = 128 * 128;      // 16 KB: span of one A operand (128 rows x 128 bytes)
constexpr int kOneThreads = 10 * 32;
constexpr uint32_t kOneTmemCols = 512;
constexpr uint32_t kColD = 0, kColSfAct = 256, kColSfW = 384;  // accumulator | scale factors of the term rows | of the weights
// The token's term rows and their scale bytes are written kCopies times (16 KB + 1 KB each at H = 4096) and CTA i reads
// copy i % kCopies: every CTA with an item fetches them at the same moment, and with a single copy each cache line is
// asked for by hundreds of requesters at once.
constexpr int kCopies = 4;

struct OneArgs {
  const float* logits;      // [E]
  const __nv_bfloat16* x;   // [H]
  __nv_bfloat16* out;       // [H]
  int* ids_out;             // [k] or null
  float* w_out;             // [k] or null
  float* part;              // [k + n_shared][I/256][H] partial sums of the down projection
  uint8_t* aq1;             // [kCopies][8][H/2] E2M1 term rows of the token, written by the CTAs that split it
  uint8_t* sf1;             // [kCopies][8][H/32] their scale bytes
  int* sync;                // counter block, zero between calls
  int* status;              // never null
  int own_status;           // the library's own status word: the last CTA clears it
  int E, H, I, k;
  int blocked;              // weights in moe_prepack's tile-contiguous layout
  int n_shared;             // 1: slot k is the shared expert (its own tensor maps, expert 0 of them), added with weight 1
  int blocked_shared;       //    and its weights' layout
};

struct OneSmem {
  uint32_t ring, a1, a2, sc, sf2, logit, route, bars, misc, total;
};
// A operand of the gate/up projection: the token's 8 term rows of one K step, 4 copies (one per lane quadrant of the
// accumulator, so that each epilogue warp finds the token in its own quadrant), fetched by TMA with every stage of the
// weight ring.  Row 32 q + t of ring stage s sits at (s / 4) * 16 KB + (s % 4) * 1 KB + q * 4 KB + t * 128: four stages
// interleave inside one 16 KB operand span, each using the 8-row group the others leave empty.  The MMA of a stage
// reads 128 rows from its own base (up to 3 KB past the span); rows it does not own hold other stages' data and feed
// accumulator lanes nobody reads.
__host__ __device__ inline uint32_t a1_slot(int s) { return static_cast<uint32_t>((s >> 2) * kATile + (s & 3) * 1024); }
__host__ __device__ inline uint32_t a1_bytes(int) { return static_cast<uint32_t>((kWStages + 3) / 4) * kATile + 4096; }
constexpr int kA2Bytes = 2048;  // B operand of the down projection: the 8 term rows of one K step (N = 16 reads 16 rows)
__host__ __device__ inline OneSmem one_smem(int E, int H) {
  OneSmem m;
  uint32_t off = 0;
  m.ring = off;
  off += kWStages * kWStage;
  m.a1 = off;
  off += a1_bytes(H);
  m.a2 = off;  // the term rows of the pair's slice of the intermediate, row t at t * 128 (1024-byte aligned)
  off += kA2Bytes;
  m.sc = off;
  off += kScStages * kScStage;
  m.sf2 = off;  // scale bytes of the intermediate's term rows for the pair's K step [8][8]
  off += 64;
  m.logit = off;
  off += (static_cast<uint32_t>(E) * 4 + 15u) & ~15u;
  m.route = off;  // ids[32], weights[32]
  off += 2 * 32 * 4;
  m.bars = off;
  off += 32 * 8;
  m.misc = off;
  off += 64;
  m.total = off;
  return m;
}

MOE_DEVINL uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in another CTA of the cluster
MOE_DEVINL uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(cta_rank));
  return r;
}
MOE_DEVINL void st_cluster_u16(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u16 [%0], %1;" ::"r"(addr), "h"(static_cast<unsigned short>(v)) : "memory");
}
MOE_DEVINL void st_cluster_u8(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u8 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
MOE_DEVINL void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
MOE_DEVINL void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }

}  // namespace

__global__ void __launch_bounds__(kOneThreads, 1)
decode_one_kernel(const __grid_constant__ CUtensorMap tmap_w13, const __grid_constant__ CUtensorMap tmap_s13,
                  const __grid_constant__ CUtensorMap tmap_w2, const __grid_constant__ CUtensorMap tmap_s2,
                  const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_sw13,
                  const __grid_constant__ CUtensorMap tmap_ss13, const __grid_constant__ CUtensorMap tmap_sw2,
                  const __grid_constant__ CUtensorMap tmap_ss2, const OneArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const OneSmem sm = one_smem(a.E, a.H);
  unsigned char* sW = smem + sm.ring;
  unsigned char* sA1 = smem + sm.a1;
  unsigned char* sA2 = smem + sm.a2;
  unsigned char* sSc = smem + sm.sc;
  unsigned char* sSf2 = smem + sm.sf2;
  float* s_logit = reinterpret_cast<float*>(smem + sm.logit);
  int* s_ids = reinterpret_cast<int*>(smem + sm.route);
  float* s_w = reinterpret_cast<float*>(s_ids + 32);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sm.bars);
  uint64_t* full_w = bars;                    // [kWStages]  TMA -> MMA
  uint64_t* empty_w = full_w + kWStages;      // [kWStages]  MMA done -> producer
  uint64_t* full_sc = empty_w + kWStages;     // [kScStages] TMA -> scale warps
  uint64_t* empty_sc = full_sc + kScStages;   // [kScStages] scale warps -> producer
  uint64_t* sf_full = empty_sc + kScStages;   // [kSfGroups] scale warps -> MMA
  uint64_t* sf_free = sf_full + kSfGroups;    // [kSfGroups] MMA done -> scale warps
  uint64_t* acc_full = sf_free + kSfGroups;   // [2, the second unused] MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;         // [2, the second unused] epilogue -> MMA
  uint64_t* act_ready = acc_empty + 2;        // epilogue warps -> MMA: an A operand and its scale factors are in place
  uint64_t* route_ready = act_ready + 1;      // routing warp -> producer
  uint64_t* split_ready = route_ready + 1;    // routing warp -> producer: the token's term rows are complete in global memory
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + sm.misc);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int grid = static_cast<int>(gridDim.x);
  const int tiles0 = a.I / 128;          // gate/up items per slot
  const int n_ks0 = a.H / 256;           // K steps of the gate/up projection
  const int npp = a.I / 256;             // K steps of the down projection = pairs of CTAs per slot
  const int n_t1 = a.H / 512;            // 256-row tiles of the down projection per CTA (half of the H rows)
  const int item = static_cast<int>(blockIdx.x);
  const int n_slots = a.k + a.n_shared;  // routed slots, then the shared expert (figure "Execution structure": it runs beside them)
  const bool has_item = item < n_slots * tiles0;
  const int slot = item / tiles0, tile = item % tiles0;
  const int pp = tile >> 1;
  const uint32_t rank = cluster_ctarank();  // = tile & 1 for a CTA with an item (tiles0 is even, clusters are (2c, 2c + 1))

#ifdef MOE_TRACE
  if (tid == 0) {
    for (int i = 0; i < 32; ++i) g_one_trace[blockIdx.x][i] = 0;
    MOE_TP(0);
  }
#endif
  // ---- set-up: barriers, tensor memory, descriptors ----
  if (tid == 32 * 3) {
    prefetch_tmap(&tmap_w13);
    prefetch_tmap(&tmap_s13);
    prefetch_tmap(&tmap_w2);
    prefetch_tmap(&tmap_s2);
    prefetch_tmap(&tmap_a1);
    if (a.n_shared) {
      prefetch_tmap(&tmap_sw13);
      prefetch_tmap(&tmap_ss13);
      prefetch_tmap(&tmap_sw2);
      prefetch_tmap(&tmap_ss2);
    }
  }
  if (tid == 0) {
    for (int s = 0; s < kWStages; ++s) { mbar_init(&full_w[s], 1); mbar_init(&empty_w[s], 1); }
    for (int s = 0; s < kScStages; ++s) { mbar_init(&full_sc[s], 1); mbar_init(&empty_sc[s], 4); }
    for (int s = 0; s < kSfGroups; ++s) { mbar_init(&sf_full[s], 4); mbar_init(&sf_free[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
    mbar_init(act_ready, 4);
    mbar_init(route_ready, 1);
    mbar_init(split_ready, 1);
    mbar_fence_init();
  }
  if (wid == 1) tmem_alloc(tmem_holder, kOneTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  pdl_launch_dependents();  // the next kernel on the stream may become resident; it waits before it touches anything
  if (tid == 0) MOE_TP(1);

  const int q = wid & 3;                         // tensor-memory lane quadrant this warp may access; also its scheduler
  const uint32_t lane_base = static_cast<uint32_t>(q * 32) << 16;
  const int jl = lane >> 3, tl = lane & 7;
  const int cb = 16 * (tl & 1) + 8 * ((tl >> 1) & 1) + 4 * (tl >> 2);  // column offset a lane ends up with (see reduce8)
  const uint32_t sA2_u = smem_u32(sA2), sSf2_u = smem_u32(sSf2);
  const int n_blk = a.H / 32;
  const int n_split_ctas = n_blk / 8;            // the first CTAs (the earliest to start) split the token row, 8 blocks each

  // Accumulator lane = term row.  A 32x32b load hands each lane 32 columns of its row; three exchange rounds over the
  // 8 lanes of the token (each halves the columns a lane keeps) leave lane t with the 8-term sums of 4 consecutive
  // columns, at offset cb of the 32.
  auto reduce8 = [&](const uint32_t (&vc)[32], float (&o)[4]) {
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
    for (int k = 0; k < 4; ++k) o[k] = ((tl & 4) ? a8[4 + k] : a8[k]) + __shfl_xor_sync(0xffffffffu, (tl & 4) ? a8[k] : a8[4 + k], 4);
  };

  // Every thread waits for the kernel launched before this one on the stream (logits and the token row may be its
  // outputs; the counter block is clear once it has completed) and looks at the two words nobody ever writes.
  pdl_wait();
  const int dirty = __ldcg(a.sync + kSyncCanary0) | __ldcg(a.sync + kSyncCanary1);
  const bool skip = dirty != 0;
  if (tid == 0) {
    MOE_TP(2);
    if (skip) atomicExch(a.status, static_cast<int>(MOE_ERR_WORKSPACE));
  }
  // The pair's one cluster barrier: every thread arrives once - here, except the epilogue warps of a CTA with an item,
  // which arrive after their stores into the partner's shared memory - and waits once before it leaves the kernel.
  if (!skip && !(has_item && wid >= 6)) cluster_arrive();

  if (skip) {
    // a counter block that was never cleared: nothing runs
  } else if (wid == 0) {
    // =========================== producer: all TMA loads of both projections ===========================
    if (lane == 0 && has_item) {
      const bool shared = slot >= a.k;  // the shared expert's weights depend on no routing: its stream starts at once
      if (!shared) mbar_wait(route_ready, 0u, a.status);
      const int e = shared ? 0 : s_ids[slot];
      const int blocked = shared ? a.blocked_shared : a.blocked;
      int s = 0, cs = 0;
      uint32_t ph = 0, cph = 0;
      const uint64_t stream_once = l2_policy_evict_first();  // every weight byte is read once per call
      for (int phase = 0; phase < 2; ++phase) {
        const CUtensorMap* mw = phase == 0 ? (shared ? &tmap_sw13 : &tmap_w13) : (shared ? &tmap_sw2 : &tmap_w2);
        const CUtensorMap* msc = phase == 0 ? (shared ? &tmap_ss13 : &tmap_s13) : (shared ? &tmap_ss2 : &tmap_s2);
        const int n_steps = phase == 0 ? n_ks0 : npp;  // K steps of the projection (tile geometry of the packed layout)
        const int n_it = phase == 0 ? n_ks0 : n_t1;
        for (int it = 0; it < n_it; ++it) {
          // gate/up: K step `it` of the item's 128 gate rows and 128 up rows; down: K step pp of row tile `it` of this
          // CTA's half of the expert's H rows
          const int ks = phase == 0 ? it : pp;
          const int wrow_a = phase == 0 ? e * 2 * a.I + tile * 128 : e * a.H + static_cast<int>(rank) * (a.H / 2) + it * kTile;
          const int wrow_b = phase == 0 ? wrow_a + a.I : wrow_a + 128;
          if (phase == 1 || (it & 1) == 0) {  // 16 scale bytes per weight row cover two K steps
            mbar_wait(&empty_sc[cs], cph ^ 1u, a.status);
            mbar_expect_tx(&full_sc[cs], kScStage);
            const int sx = blocked ? 0 : (ks >> 1) * 16;
            const int sya = blocked ? ((wrow_a >> 7) * (n_steps >> 1) + (ks >> 1)) * 128 : wrow_a;
            const int syb = blocked ? ((wrow_b >> 7) * (n_steps >> 1) + (ks >> 1)) * 128 : wrow_b;
            tma_load_2d_hint(sSc + cs * kScStage, msc, sx, sya, &full_sc[cs], stream_once);
            tma_load_2d_hint(sSc + cs * kScStage + 128 * 16, msc, sx, syb, &full_sc[cs], stream_once);
            if (++cs == kScStages) { cs = 0; cph ^= 1u; }
          }
          mbar_wait(&empty_w[s], ph ^ 1u, a.status);
          mbar_expect_tx(&full_w[s], phase == 0 ? kWStage + 4 * 1024 : kWStage);
          const int wx = blocked ? 0 : ks * 128;
          const int wya = blocked ? ((wrow_a >> 7) * n_steps + ks) * 128 : wrow_a;
          const int wyb = blocked ? ((wrow_b >> 7) * n_steps + ks) * 128 : wrow_b;
          tma_load_2d_hint(sW + s * kWStage, mw, wx, wya, &full_w[s], stream_once);
          tma_load_2d_hint(sW + s * kWStage + 128 * 128, mw, wx, wyb, &full_w[s], stream_once);
          if (it == 0) MOE_TP(5 + phase);
          if (phase == 0) {
            if (it == 0) {  // the weights depend on the routing alone; the token's term rows on the CTAs that split it
              mbar_wait(split_ready, 0u, a.status);
              fence_proxy_async_all();  // the rows were written through the generic proxy, TMA reads through the async one
              MOE_TP(20);
            }
#pragma unroll
            for (int qq = 0; qq < 4; ++qq)
              tma_load_2d(sA1 + a1_slot(s) + qq * 4096, &tmap_a1, ks * 128, (item % kCopies) * kTerms, &full_w[s]);
          }
          if (++s == kWStages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (wid == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0 && has_item) {
      int s = 0, slotg = 0;
      uint32_t ph = 0, sph = 0;
      const uint32_t d_addr = tmem_base + kColD;
      // ---- gate/up: one accumulator over all K steps ----
      mbar_wait(act_ready, 0u, a.status);
      tc_fence_after_sync();
      MOE_TP(21);
      for (int ks = 0; ks < n_ks0; ++ks) {
        if ((ks & 1) == 0) mbar_wait(&sf_full[slotg], sph, a.status);
        if (ks == 0) MOE_TP(22);
        mbar_wait(&full_w[s], ph, a.status);
        tc_fence_after_sync();
        if (ks == 0) MOE_TP(7);
        const uint32_t w_addr = smem_u32(sW + s * kWStage);
        const uint32_t a_addr = smem_u32(sA1) + a1_slot(s);
#pragma unroll
        for (uint32_t j = 0; j < 4; ++j) {  // K = 64 each; scale word (ks & 1) * 2 + j / 2 of the group, half j & 1
          const uint32_t sf_act = tmem_base + kColSfAct + static_cast<uint32_t>(ks * 8) + (j >> 1) * 4;
          const uint32_t sf_w = tmem_base + kColSfW + static_cast<uint32_t>(slotg * 32 + ((ks & 1) * 2 + (j >> 1)) * 8);
          umma_mxf4(d_addr, umma_desc_k_sw128(a_addr + j * 32), umma_desc_k_sw128(w_addr + j * 32), idesc_mxf4(j & 1u), sf_act,
                    sf_w, (ks | static_cast<int>(j)) != 0 ? 1u : 0u);
        }
        umma_commit(&empty_w[s]);
        if (++s == kWStages) { s = 0; ph ^= 1u; }
        if ((ks & 1) == 1) {
          umma_commit(&sf_free[slotg]);
          if (++slotg == kSfGroups) { slotg = 0; sph ^= 1u; }
        }
      }
      umma_commit(&acc_full[0]);
      MOE_TP(8);
      // ---- down: a single K step.  The operands change places: the 128 weight rows of a sub-tile are the M side, the
      // 8 term rows of the pair's slice the N side (N = 16, the smallest; its upper 8 rows are never looked at), so the
      // accumulator of a sub-tile is 16 columns and those of all H/256 sub-tiles of this CTA sit side by side in the
      // 256 columns: no accumulator is handed back and forth with the epilogue, which reads them all once at the end ----
      mbar_wait(act_ready, 1u, a.status);
      mbar_wait(&acc_empty[0], 0u, a.status);  // the gate/up accumulator has been read
      tc_fence_after_sync();
      MOE_TP(9);
      const uint32_t a2_addr = smem_u32(sA2);
      for (int n = 0; n < n_t1; ++n) {
        mbar_wait(&sf_full[slotg], sph, a.status);
        mbar_wait(&full_w[s], ph, a.status);
        tc_fence_after_sync();
#pragma unroll
        for (uint32_t b = 0; b < 2; ++b) {
          const uint32_t w_addr = smem_u32(sW + s * kWStage) + b * (128u * 128u);
#pragma unroll
          for (uint32_t j = 0; j < 4; ++j) {
            const uint32_t sf_act = tmem_base + kColSfAct + (j >> 1) * 4;
            const uint32_t sf_w = tmem_base + kColSfW + static_cast<uint32_t>(slotg * 32 + ((pp & 1) * 2 + static_cast<int>(j >> 1)) * 8) + b * 4;
            umma_mxf4(d_addr + static_cast<uint32_t>(2 * n) * 16u + b * 16u, umma_desc_k_sw128(w_addr + j * 32),
                      umma_desc_k_sw128(a2_addr + j * 32), idesc_mxf4(j & 1u, 16u), sf_w, sf_act, j != 0 ? 1u : 0u);
          }
        }
        umma_commit(&empty_w[s]);
        umma_commit(&sf_free[slotg]);
        if (++s == kWStages) { s = 0; ph ^= 1u; }
        if (++slotg == kSfGroups) { slotg = 0; sph ^= 1u; }
      }
      umma_commit(&acc_full[0]);
      MOE_TP(10);
    }
  } else {
    // =========================== warps 2..9 ===========================
    // ---- warp 8 routes: top-k by logit (ties to the lower expert), softmax over the selected logits ----
    if (wid == 8) {
      for (int e0 = 0; e0 < a.E; e0 += 256) {  // eight loads in flight per lane
        float lv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int e = e0 + 32 * u + lane;
          lv[u] = e < a.E ? __ldg(a.logits + e) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int e = e0 + 32 * u + lane;
          if (e < a.E) s_logit[e] = lv[u];
        }
      }
      __syncwarp();
      if (lane == 0) MOE_TP(3);
      int my_id;
      float my_v;
      warp_topk(s_logit, a.E, a.k, lane, &my_id, &my_v);
      const float wt = warp_softmax_selected(my_v, a.k, lane);
      if (lane < a.k) {
        s_ids[lane] = my_id;
        s_w[lane] = wt;
        if (blockIdx.x == 0 && a.ids_out != nullptr) a.ids_out[lane] = my_id;
        if (blockIdx.x == 0 && a.w_out != nullptr) a.w_out[lane] = wt;
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(route_ready);  // the producer reads its expert; the reduction reads the weights much later
        MOE_TP(4);
      }
    }
    // ---- the token row -> 8 E2M1 term rows.  Splitting the whole row in every CTA would cost several microseconds of
    // issue time (eight dependent terms for each of H/32 blocks), so the first H/256 CTAs - the earliest to start -
    // split 8 blocks of 32 elements each (warps 6 and 9, one block per group of 8 lanes, about a microsecond), store
    // the codes and scale bytes to global memory and count themselves in; every CTA with an item then fetches the
    // rows K step by K step with its weight stages (TMA, from L2; four copies of each row) ----
    if ((wid == 6 || wid == 9) && item < n_split_ctas) {
      const int b = item * 8 + (wid == 9 ? 4 : 0) + jl;
      const uint2 v = __ldg(reinterpret_cast<const uint2*>(a.x + b * 32 + tl * 4));
      float r[1][4] = {{__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u), __uint_as_float(v.y << 16),
                       __uint_as_float(v.y & 0xFFFF0000u)}};
      split_terms<1>(r, [&](int, int t, uint32_t bytes, int se) {
#pragma unroll
        for (int cp = 0; cp < kCopies; ++cp) {
          *reinterpret_cast<uint16_t*>(a.aq1 + (static_cast<size_t>(cp) * kTerms + t) * (a.H / 2) + b * 16 + tl * 2) = static_cast<uint16_t>(bytes);
          if (tl == 0) a.sf1[(static_cast<size_t>(cp) * kTerms + t) * n_blk + b] = static_cast<uint8_t>(se + 127);
        }
      });
      __syncwarp();  // orders the lanes' stores before lane 0's release
      if (lane == 0) {
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.sync + kSyncSplit) : "memory");
        MOE_TP(24);
      }
    }
    if (has_item && wid == 8) {
      // the routing warp waits for the split and tells the producer (whose TMA loads bring the term rows in with the
      // weight stages) and the epilogue warps (which fetch the rows' scale bytes).  All 32 lanes poll the same word: a
      // warp whose lane 0 has gone through a long loop of its own runs the warp-wide code after it several times slower
      counter_wait_ge(a.sync + kSyncSplit, 2 * n_split_ctas, a.status);
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(split_ready);
        MOE_TP(25);
      }
    }
    if (wid < 6) {
      // =========================== weight scale bytes: shared memory -> tensor memory ===========================
      if (has_item) {
        int cs = 0, slotg = 0;
        uint32_t cph = 0, sfree_ph = 0;
        const int n_sc = n_ks0 / 2 + n_t1;  // scale stages of the gate/up K steps (two per stage), then one per down tile
        for (int i = 0; i < n_sc; ++i) {
          mbar_wait(&full_sc[cs], cph, a.status);
          mbar_wait(&sf_free[slotg], sfree_ph ^ 1u, a.status);
          __syncwarp();  // the waits may leave lanes diverged; tcgen05.st is warp-collective
          const unsigned char* blk = sSc + cs * kScStage;
          uint4 r[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) r[c] = *reinterpret_cast<const uint4*>(blk + (lane + 32 * c) * 16);
          // column 8t + c of the group: scale word t (K blocks 4t..4t+3 of the 16) for weight row lane + 32c
          asm volatile(
              "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
              "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(
                  tmem_base + lane_base + kColSfW + static_cast<uint32_t>(slotg * 32)),
              "r"(r[0].x), "r"(r[1].x), "r"(r[2].x), "r"(r[3].x), "r"(r[4].x), "r"(r[5].x), "r"(r[6].x), "r"(r[7].x),
              "r"(r[0].y), "r"(r[1].y), "r"(r[2].y), "r"(r[3].y), "r"(r[4].y), "r"(r[5].y), "r"(r[6].y), "r"(r[7].y),
              "r"(r[0].z), "r"(r[1].z), "r"(r[2].z), "r"(r[3].z), "r"(r[4].z), "r"(r[5].z), "r"(r[6].z), "r"(r[7].z),
              "r"(r[0].w), "r"(r[1].w), "r"(r[2].w), "r"(r[3].w), "r"(r[4].w), "r"(r[5].w), "r"(r[6].w), "r"(r[7].w)
              : "memory");
          tmem_st_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(&sf_full[slotg]);
            mbar_arrive(&empty_sc[cs]);
          }
          if (++cs == kScStages) { cs = 0; cph ^= 1u; }
          if (++slotg == kSfGroups) { slotg = 0; sfree_ph ^= 1u; }
        }
      }
    } else if (has_item) {
      // =========================== epilogue warps ===========================
      // ---- scale factors of the token's term rows -> tensor memory: K step ks owns two scale-factor blocks (its two
      // scale words); column c of a block holds, in lane l of every quadrant, the word of operand row 32c + l, which
      // for every c is term row l & 7 (the four copies).  Four K steps per store. ----
      __syncwarp();
      mbar_wait(split_ready, 0u, a.status);  // the first CTAs have written the scale bytes (and the rows) of the token's terms
      __syncwarp();
      if (wid == 6 && lane == 0) MOE_TP(11);
      {
        // lane l needs the H/32 scale bytes of term row l & 7: all loads first (one L2 round trip), then the stores
        constexpr int kMaxVec = 4096 / 32 / 16;  // 8 pieces of 16 bytes at H = 4096
        uint4 sv[kMaxVec];
        const uint8_t* srow = a.sf1 + (static_cast<size_t>(item % kCopies) * kTerms + tl) * n_blk;
#pragma unroll
        for (int i = 0; i < kMaxVec; ++i)
          if (i * 16 < n_blk) sv[i] = __ldcg(reinterpret_cast<const uint4*>(srow + i * 16));
#pragma unroll
        for (int i = 0; i < kMaxVec; i += 2) {  // 32 scale bytes = 4 K steps per store
          if (i * 16 < n_blk) {
            const uint4 lo = sv[i], hi = sv[i + 1];  // (n_blk is a multiple of 16; a missing upper half is never used)
            const uint32_t x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};  // word pairs of K steps 2i .. 2i+3
            uint32_t w[32];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                w[u * 8 + c] = x[2 * u];
                w[u * 8 + 4 + c] = x[2 * u + 1];
              }
            asm volatile(
                "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(
                    tmem_base + lane_base + kColSfAct + static_cast<uint32_t>(i * 16)),
                "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "r"(w[8]), "r"(w[9]),
                "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15]), "r"(w[16]), "r"(w[17]), "r"(w[18]),
                "r"(w[19]), "r"(w[20]), "r"(w[21]), "r"(w[22]), "r"(w[23]), "r"(w[24]), "r"(w[25]), "r"(w[26]), "r"(w[27]),
                "r"(w[28]), "r"(w[29]), "r"(w[30]), "r"(w[31])
                : "memory");
          }
        }
      }
      tmem_st_wait();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(act_ready);
      if (wid == 6 && lane == 0) MOE_TP(12);

      float* prow = a.part + (static_cast<size_t>(slot) * npp + pp) * a.H + static_cast<size_t>(rank) * (a.H / 2);
      const uint32_t chunk = rank * 4u + static_cast<uint32_t>(q);
      const uint32_t peer_a2 = map_to_cta(sA2_u, rank ^ 1u), peer_sf2 = map_to_cta(sSf2_u, rank ^ 1u);
      // Sweep 0 runs the two epilogues "dry" - the same instructions on whatever tensor memory holds, with every wait,
      // signal and store left out - while the first accumulator fills: each CTA executes this code only once or a few
      // times, and its first real use, which is on the critical path, would otherwise pay for fetching it.
      for (int sweep = 0; sweep < 2; ++sweep) {
        const bool dry = sweep == 0;
        // ---- gate/up accumulator: gate chunk q and up chunk 4 + q of the 8 chunks of 32 columns ----
        if (!dry) {
          mbar_wait(&acc_full[0], 0u, a.status);
          if (wid == 6 && lane == 0) MOE_TP(13);
        }
        __syncwarp();  // tcgen05.ld is warp-collective
        tc_fence_after_sync();
        float gsel[4], usel[4];
        {
          uint32_t vg[32], vu[32];
          tmem_ld_32x32(tmem_base + lane_base + kColD + static_cast<uint32_t>(32 * q), vg);
          tmem_ld_32x32(tmem_base + lane_base + kColD + static_cast<uint32_t>(32 * (4 + q)), vu);
          tmem_ld_wait();
          tc_fence_before_sync();
          __syncwarp();
          if (!dry && lane == 0) mbar_arrive(&acc_empty[0]);  // the accumulator is free for the down projection
          reduce8(vg, gsel);
          reduce8(vu, usel);
        }
        {
          // SwiGLU, bf16 rounding (the intermediate is defined as a bf16 value) and the 8-term split of this warp's block
          // of 32: block q of this CTA's four = 16-byte chunk rank * 4 + q of the pair's 128-byte K step.  The rows go
          // to this CTA's operand and to the partner's.
          float r[1][4];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float sv = __fdividef(gsel[c], 1.0f + __expf(-gsel[c])) * usel[c];
            r[0][c] = __bfloat162float(__float2bfloat16_rn(sv));
          }
          const bool live = !dry && jl == 0;
          split_terms<1>(r, [&](int, int t, uint32_t bytes, int se) {
            if (live) {
              const uint32_t off = static_cast<uint32_t>(t * 128) + ((chunk ^ static_cast<uint32_t>(t)) << 4) + static_cast<uint32_t>(cb >> 1);
              asm volatile("st.shared.u16 [%0], %1;" ::"r"(sA2_u + off), "h"(static_cast<unsigned short>(bytes)) : "memory");
              st_cluster_u16(peer_a2 + off, bytes);
              if (tl == 0) {
                sSf2[t * 8 + static_cast<int>(chunk)] = static_cast<uint8_t>(se + 127);
                st_cluster_u8(peer_sf2 + static_cast<uint32_t>(t * 8) + chunk, static_cast<uint32_t>(se + 127));
              }
            }
          });
        }
        if (!dry) {
          if (wid == 6 && lane == 0) MOE_TP(14);
          fence_proxy_async_all();  // both CTAs' tensor cores read these rows through the asynchronous proxy
          __syncwarp();
          cluster_arrive();
          cluster_wait();  // the partner's rows and scale bytes are in this CTA's shared memory
          fence_proxy_async_smem();
          if (wid == 6 && lane == 0) MOE_TP(15);
        }
        {
          const uint2 v = *reinterpret_cast<const uint2*>(sSf2 + tl * 8);
          const uint32_t w[8] = {v.x, v.x, v.x, v.x, v.y, v.y, v.y, v.y};
          if (!dry) {
            tmem_st_32x8(tmem_base + lane_base + kColSfAct, w);
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(act_ready);
          }
        }
        // ---- down accumulators, all sub-tiles at once: lane = weight row of the sub-tile, 16 columns per sub-tile of
        // which the first 8 are the 8 terms; their sum, in ascending term order, is the row's partial sum ----
        if (!dry) mbar_wait(&acc_full[0], 1u, a.status);
        __syncwarp();
        tc_fence_after_sync();
        for (int u0 = 0; u0 < (dry ? 2 : 2 * n_t1); u0 += 2) {  // two sub-tiles (32 columns) per load
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + lane_base + kColD + static_cast<uint32_t>(u0 * 16), v);
          tmem_ld_wait();
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float sum = __uint_as_float(v[16 * h]);
#pragma unroll
            for (int t = 1; t < kTerms; ++t) sum = __fadd_rn(sum, __uint_as_float(v[16 * h + t]));
            if (!dry) prow[(u0 + h) * 128 + 32 * q + lane] = sum;
          }
        }
        tc_fence_before_sync();
        if (!dry) {
          // one release for all of this warp's stores (a release per tile would wait a memory round trip each time),
          // counted for this CTA's half of the output columns
          __syncwarp();
          if (lane == 0)
            asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.sync + kSyncDone2 + static_cast<int>(rank)) : "memory");
          if (wid == 6 && lane == 0) MOE_TP(16);
        }
      }
    }
  }

  // ---- no CTA leaves while its partner may still write to its shared memory: every thread that arrived at the pair's
  // cluster barrier above waits for it here (the epilogue warps of a CTA with an item did both after their stores) ----
  __syncthreads();
  if (!skip && !(has_item && wid >= 6)) cluster_wait();

  // ---- reduction: the last H/128 CTAs own 128 output columns each ----
  constexpr int kRedCols = 128;
  const int n_red = a.H / kRedCols;
  const int ct = item - (grid - n_red);
  // y_j[n] = sum over p ascending of part[j][p][n]; out[n] = bf16(fma chain over j = 0..k-1 from zero)
  auto reduce_tile = [&](const bool dry) {
    float* ys = reinterpret_cast<float*>(sW);  // [k][128], the ring is idle by now
    const int cg = tid & 31, grp = tid >> 5;   // 32 groups of 4 columns; warp j sums the partials of slot j, j + 8, ...
    if (grp < 8) {
      for (int j = grp; j < n_slots; j += 8) {
        const float* p0 = a.part + static_cast<size_t>(j) * npp * a.H + ct * kRedCols + cg * 4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int p = 0; p < npp; p += 8) {  // eight independent 16-byte loads in flight
          float4 v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (p + u < npp) v[u] = __ldcg(reinterpret_cast<const float4*>(p0 + static_cast<size_t>(p + u) * a.H));
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (p + u < npp) {
              if (p + u == 0) {
                acc = v[u];
              } else {
                acc.x = __fadd_rn(acc.x, v[u].x); acc.y = __fadd_rn(acc.y, v[u].y);
                acc.z = __fadd_rn(acc.z, v[u].z); acc.w = __fadd_rn(acc.w, v[u].w);
              }
            }
        }
        *reinterpret_cast<float4*>(ys + j * kRedCols + cg * 4) = acc;
      }
    }
    __syncthreads();
    if (tid < kRedCols / 2) {
      const int col = tid * 2;
      float2 acc = make_float2(0.0f, 0.0f);
      for (int j = 0; j < a.k; ++j) {
        const float wj = s_w[j];
        const float2 v = *reinterpret_cast<const float2*>(ys + j * kRedCols + col);
        acc.x = __fmaf_rn(wj, v.x, acc.x);
        acc.y = __fmaf_rn(wj, v.y, acc.y);
      }
      if (a.n_shared) {  // the join: one fp32 addition of the shared expert's row after the routed slots' recurrence
        const float2 v = *reinterpret_cast<const float2*>(ys + a.k * kRedCols + col);
        acc.x = __fadd_rn(acc.x, v.x);
        acc.y = __fadd_rn(acc.y, v.y);
      }
      if (!dry) *reinterpret_cast<__nv_bfloat162*>(a.out + ct * kRedCols + col) = __floats2bfloat162_rn(acc.x, acc.y);
    }
    __syncthreads();
  };
  if (!skip) {
    if (ct >= 0) {
      reduce_tile(true);  // once on whatever the buffer holds, no store: the code is then in place when the count completes
      if (tid == 0) {
        counter_wait_ge(a.sync + kSyncDone2 + (2 * ct) / n_red, 4 * n_slots * npp, a.status);  // the half its columns are in
        MOE_TP(17);
      }
      __syncthreads();
    }
    // this CTA's last access to the counters is behind it: it counts itself out, and the last CTA to do so clears the
    // block for the next call (beside the arithmetic below, not after it)
    if (tid == 0) {
      __threadfence();
      if (atomicAdd(a.sync + kSyncExit, 1) == grid - 1) {
        __threadfence();
        a.sync[kSyncDone2] = 0;
        a.sync[kSyncDone2 + 1] = 0;
        a.sync[kSyncExit] = 0;
        a.sync[kSyncSplit] = 0;
        if (a.own_status) *a.status = 0;
      }
    }
    if (ct >= 0) {
      reduce_tile(false);
      if (tid == 0) MOE_TP(18);
    }
  }

  // ---- teardown ----
  tc_fence_before_sync();
  __syncthreads();
  if (wid == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kOneTmemCols);
  }
  if (tid == 0) MOE_TP(19);
}

// ---- host side ---------------------------------------------------------------------------------------
// Shapes: one token; H and I multiples of 512 up to 4096 (whole 256-row tiles, whole pairs); one gate/up item and one
// reducing CTA per SM at most; the routing row and the operands fit shared memory.
bool decode_one_ok(const moe_shape_t& sh, const void* w13, const void* w2, int n_shared) {
  const int grid = sm_count() & ~1;
  return sh.T == 1 && sh.H % 512 == 0 && sh.I % 512 == 0 && sh.H <= 4096 && sh.I <= 4096 && sh.k <= 32 &&
         (sh.k + n_shared) * (sh.I / 128) <= grid && sh.H / 32 <= grid && sh.H / 128 <= grid && sh.H / 256 <= kSyncExit - kSyncDone2 &&
         (reinterpret_cast<uintptr_t>(w13) & 15u) == 0 && (reinterpret_cast<uintptr_t>(w2) & 15u) == 0 &&
         one_smem(sh.E, sh.H).total + 1024 <= 227 * 1024;
}
size_t decode_one_scratch_bytes(const moe_shape_t& sh, int n_shared) {
  return align_up(static_cast<size_t>(sh.k + n_shared) * (sh.I / 256) * sh.H * 4, kAlign) +
         align_up(static_cast<size_t>(kCopies) * kTerms * (sh.H / 2), kAlign) + align_up(static_cast<size_t>(kCopies) * kTerms * (sh.H / 32), kAlign);
}

int launch_decode_one(const float* logits, const __nv_bfloat16* x, const ExpertWeights& w, const moe_shape_t& sh,
                      __nv_bfloat16* out, int* ids_out, float* w_out, int* sync, void* scratch, StatusRef status,
                      cudaStream_t st, const ExpertWeights* shared) {
  static PerDeviceFlag flag;
  if (!once_per_device(flag, [] {
        return cudaFuncSetAttribute(decode_one_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess;
      }))
    return MOE_ERR_CUDA;
  CUtensorMap tm_w13, tm_w2, tm_s13, tm_s2;
  if (!weight_maps(w, sh, &tm_w13, &tm_s13, &tm_w2, &tm_s2)) return MOE_ERR_CUDA;
  // the shared expert, where there is one: tensors shaped as the routed ones with a single expert
  CUtensorMap tm_sw13 = tm_w13, tm_sw2 = tm_w2, tm_ss13 = tm_s13, tm_ss2 = tm_s2;
  const int n_shared = shared != nullptr ? 1 : 0;
  if (shared != nullptr && !weight_maps(*shared, moe_shape_t{1, sh.H, sh.I, 1, 1}, &tm_sw13, &tm_ss13, &tm_sw2, &tm_ss2)) return MOE_ERR_CUDA;
  OneArgs a;
  a.logits = logits;
  a.x = x;
  a.out = out;
  a.ids_out = ids_out;
  a.w_out = w_out;
  a.part = static_cast<float*>(scratch);
  a.aq1 = static_cast<uint8_t*>(scratch) + align_up(static_cast<size_t>(sh.k + n_shared) * (sh.I / 256) * sh.H * 4, kAlign);
  a.sf1 = a.aq1 + align_up(static_cast<size_t>(kCopies) * kTerms * (sh.H / 2), kAlign);
  a.sync = sync;
  a.status = status.word;
  a.own_status = status.own ? 1 : 0;
  a.E = sh.E;
  a.H = sh.H;
  a.I = sh.I;
  a.k = sh.k;
  a.blocked = w.blocked ? 1 : 0;
  a.n_shared = n_shared;
  a.blocked_shared = (shared != nullptr && shared->blocked) ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(sm_count() & ~1));
  cfg.blockDim = dim3(kOneThreads);
  cfg.dynamicSmemBytes = one_smem(sh.E, sh.H).total + 1024;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  CUtensorMap tm_a1;  // the token's 8 term rows [8][H/2 bytes], one box = 8 rows x one K step
  if (!term_row_map(&tm_a1, a.aq1, sh.H / 2, kCopies * kTerms, 8)) return MOE_ERR_CUDA;
  if (cudaLaunchKernelEx(&cfg, decode_one_kernel, tm_w13, tm_s13, tm_w2, tm_s2, tm_a1, tm_sw13, tm_ss13, tm_sw2, tm_ss2, a) != cudaSuccess)
    return MOE_ERR_CUDA;
  note_kernel(n_shared ? "block_one_launch_mxf4_pair_split_k" : "layer_one_launch_mxf4_pair_split_k", 1);
  return MOE_OK;
}

}  // namespace moe

#ifdef MOE_TRACE
extern "C" int moe_debug_trace_one(unsigned long long* out) {
  return cudaMemcpyFromSymbol(out, moe::g_one_trace, sizeof(moe::g_one_trace)) == cudaSuccess ? 0 : 1;
}
#endif
