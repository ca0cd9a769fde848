// Shared declarations of the sm_100a routed-MoE library (internal; the public ABI is include/moe_b200.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/moe_b200.h"
#include "../../include/moe_b200_debug.h"

#define MOE_DEVINL __device__ __forceinline__

namespace moe {

// ---- workspace carving (host) ----------------------------------------------------------------
// ws = [ route counters (always first) | act bf16 [S,I] | permute block counts | ffn counters ]
struct WsLayout {
  size_t act_off, route_off, permute_off, ffn_off, total;
};

constexpr int kPermuteChunk = 1024;  // slots per CTA in the multi-CTA permute
constexpr size_t kAlign = 256;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// native block-scaled FP4 variant (decode-sized batches): on average at most 32 rows per expert (2 passes of 16
// tokens over the weight stream).  Its scratch holds the E2M1 term rows (8 per row) of both projections' inputs:
// [8S, I/2] + [8S, I/32] scale bytes and [8S, H/2] + [8S, H/32]; and one completion counter per expert.
#ifndef MOE_NATIVE_MAX_SLOTS
#define MOE_NATIVE_MAX_SLOTS 6144            // measured crossover to the prefill-sized kernel at the production shape
#endif
#ifndef MOE_NATIVE_MAX_ROWS_PER_EXPERT
#define MOE_NATIVE_MAX_ROWS_PER_EXPERT 32    // on average: two passes of 16 tokens over an expert's weights
#endif
inline bool native_batch_ok(const moe_shape_t& s) {
  const long long S = static_cast<long long>(s.T) * s.k;
  return S <= MOE_NATIVE_MAX_SLOTS && S <= static_cast<long long>(MOE_NATIVE_MAX_ROWS_PER_EXPERT) * s.E;
}
inline size_t native_scratch_bytes(const moe_shape_t& s) {
  const size_t S = static_cast<size_t>(s.T) * s.k;
  return align_up(8 * S * (s.I / 2), kAlign) + align_up(8 * S * (s.I / 32), kAlign) + align_up(8 * S * (s.H / 2), kAlign) +
         align_up(8 * S * (s.H / 32), kAlign) + align_up(static_cast<size_t>(s.E) * 4, kAlign);
}

// scratch of the quantised-activation variant: one operand row per sorted row (codes and scale bytes of the token rows
// and of the intermediate) and the per-expert counters
inline size_t native_q_scratch_bytes(const moe_shape_t& s) {
  const size_t S = static_cast<size_t>(s.T) * s.k;
  return align_up(S * (s.I / 2), kAlign) + align_up(S * (s.I / 32), kAlign) + align_up(S * (s.H / 2), kAlign) +
         align_up(S * (s.H / 32), kAlign) + align_up(static_cast<size_t>(s.E) * 4, kAlign);
}

inline WsLayout ws_layout(const moe_shape_t& s) {
  WsLayout L;
  const size_t S = static_cast<size_t>(s.T) * s.k;
  size_t off = 0;
  L.route_off = off;  // moe_route is given only (T, E, k): its block must not depend on H or I
  off += align_up((static_cast<size_t>(s.E) + 8) * 4, kAlign);
  L.act_off = off;  // bf16 act[S,I], or the scratch of the native variant
  const size_t act_bytes = align_up(S * s.I * 2, kAlign);
  const size_t nat_bytes = native_batch_ok(s) ? native_scratch_bytes(s) : 0;
  off += (act_bytes > nat_bytes ? act_bytes : nat_bytes) + kAlign;
  L.permute_off = off;
  const size_t nblk = (S + kPermuteChunk - 1) / kPermuteChunk;
  off += align_up(nblk * s.E * 4, kAlign);
  L.ffn_off = off;
  off += align_up(1024, kAlign);
  L.total = off;
  return L;
}

// ---- expert weights as the kernels see them --------------------------------------------------------
// Either the checkpoint's logical layout (rows of H/2 or I/2 packed bytes, rows of K/32 scale bytes), or the layout
// moe_prepack writes for shapes with H and I multiples of 512: the same bytes in tiles that are contiguous in memory,
//   codes:  tile (row / 128, byte / 128) = [128 rows][128 bytes], tiles of one row block consecutive along K
//   scales: tile (row / 128, byte / 16)  = [128 rows][16 bytes]
// so that what a CTA fetches per pipeline step (128 rows x 128 bytes of codes, 128 rows x 16 scale bytes) is one
// contiguous 16 KB / 2 KB run instead of 128 pieces 2 KB apart: DRAM pages are read whole (the decode_c64 expert-FFN
// call went from 0.516 to 0.48 ms on the same bytes).
struct ExpertWeights {
  const uint8_t *w13, *s13, *w2, *s2;
  bool blocked;
};
inline bool blocked_shape(const moe_shape_t& s) { return s.H % 512 == 0 && s.I % 512 == 0; }
struct PackedLayout {
  size_t w13, s13, w2, s2, total;
};
inline PackedLayout packed_layout(const moe_shape_t& s) {
  PackedLayout L;
  const size_t n = static_cast<size_t>(s.E) * s.H * s.I;  // weights of one projection pair half: E * H * I
  size_t off = 0;
  L.w13 = off;
  off += align_up(n, kAlign);        // E * 2I * H/2
  L.s13 = off;
  off += align_up(n / 16, kAlign);   // E * 2I * H/32
  L.w2 = off;
  off += align_up(n / 2, kAlign);    // E * H * I/2
  L.s2 = off;
  off += align_up(n / 32, kAlign);   // E * H * I/32
  L.total = off;
  return L;
}
int launch_prepack(const uint8_t* w13, const uint8_t* s13, const uint8_t* w2, const uint8_t* s2, const moe_shape_t& s,
                   uint8_t* packed, cudaStream_t st);

// ---- the status word the kernels report through (host) ---------------------------------------------
// The caller's, or - when the caller passed NULL - one word inside the library image per device, so that the rule
// "once one bounded wait has run out, every later wait of the grid gives up after a short spin" holds for every
// call: without a word to look at, one lost signal would cost the full limit in every wait that follows it.
// The library's own word is cleared by the call that uses it (`own` tells the launcher to arrange that: by a kernel
// of the call where one runs before the waits or after them, else by a memset node before the launches); nobody
// reads it on the host.  Calls that pass NULL and overlap on the GPU share it: a timeout in one may cut short the
// waits of the other, whose results are then reported nowhere - pass a status word to know.
struct StatusRef {
  int* word;
  bool own;
};
int resolve_status(int32_t* user_word, StatusRef* out);  // MOE_OK or MOE_ERR_CUDA

// ---- per-thread call record (host) -----------------------------------------------------------
void note_kernel(const char* name, int launches);

// ---- launchers implemented in the .cu files --------------------------------------------------
int launch_route(const float* logits, int T, int E, int k, int* ids, float* w, int* offsets, int* counters,
                 cudaStream_t st);
int launch_permute(const __nv_bfloat16* x, const int* ids, const int* offsets, const moe_shape_t& s,
                   __nv_bfloat16* x_perm, int* perm, int* inv_perm, int* block_counts, cudaStream_t st,
                   const int* range_lo = nullptr, const int* range_hi = nullptr);
// weight-streaming variant (any shape; the one for decode-sized batches)
int launch_expert_ffn_stream(const __nv_bfloat16* x_perm, const int* offsets, const uint8_t* w13, const uint8_t* s13,
                             const uint8_t* w2, const uint8_t* s2, const moe_shape_t& s, __nv_bfloat16* act, float* y_perm,
                             int* status_word, cudaStream_t st, float* const* row_dst = nullptr);
// tcgen05 grouped-GEMM variant (prefill-sized batches); umma_shape_ok says whether it applies
bool umma_shape_ok(const moe_shape_t& s);
int launch_expert_ffn_umma(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& s,
                           __nv_bfloat16* act, float* y_perm, int* status_word, cudaStream_t st, float* const* row_dst = nullptr);
int launch_combine(const float* y_perm, const int* inv_perm, const float* w, const moe_shape_t& s,
                   __nv_bfloat16* out, cudaStream_t st);
int launch_validate_scales(const uint8_t* scales, size_t n, int* bad, cudaStream_t st);

// native block-scaled FP4 variant; scratch of native_scratch_bytes
bool native_shape_ok(const moe_shape_t& s, const void* w13, const void* w2);
// the quantised-activation variant of the same kernel: any batch size; scratch of native_q_scratch_bytes
bool native_q_shape_ok(const moe_shape_t& s, const void* w13, const void* w2);
int launch_expert_ffn_native_q(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& s,
                               void* scratch, float* y_perm, StatusRef status, cudaStream_t st, float* const* row_dst = nullptr);
int launch_expert_ffn_native(const __nv_bfloat16* x_perm, const int* offsets, const ExpertWeights& w, const moe_shape_t& s,
                             void* scratch, float* y_perm, StatusRef status, cudaStream_t st, float* const* row_dst = nullptr);

// the whole layer in one launch, for a handful of tokens on shapes the native variant takes (moe_forward);
// `sync` is the zeroed block of kForwardSyncBytes, `scratch` holds forward_fused_scratch_bytes
constexpr size_t kForwardSyncBytes = 8192;
// int indices inside that block (both one-launch kernels): [0, E) per-expert counters of the general kernel, then
constexpr int kSyncDone2 = 1024;      // per column tile of the output: warps that have stored their rows of a down item
constexpr int kSyncExit = 1024 + 64;  // CTAs that are through with the counters; the last one clears the block
constexpr int kSyncSplit = 1024 + 65; // general kernel: CTAs that have written their share of the tokens' term rows
// two words that no kernel ever writes: a call that finds one of them non-zero was given a block that was never
// cleared, reports MOE_ERR_WORKSPACE through the status word and does nothing (every CTA takes the same decision)
constexpr int kSyncCanary0 = 1024 + 66, kSyncCanary1 = 2047;
bool forward_fused_ok(const moe_shape_t& s, const void* w13, const void* w2);  // the kernel can take the shape
bool forward_fused_preferred(const moe_shape_t& s);                             // and is the faster choice (measured)
size_t forward_fused_scratch_bytes(const moe_shape_t& s);
int launch_forward_fused(const float* logits, const __nv_bfloat16* x, const ExpertWeights& w, const moe_shape_t& s,
                         __nv_bfloat16* out, int* ids_out, float* w_out, int* sync, void* scratch, StatusRef status,
                         cudaStream_t st);

// the whole layer for one token in one launch with the down projection split along K over pairs of CTAs (moe_forward
// at T = 1 where the shape allows it); `sync` as above, `scratch` holds decode_one_scratch_bytes
bool decode_one_ok(const moe_shape_t& s, const void* w13, const void* w2, int n_shared = 0);
size_t decode_one_scratch_bytes(const moe_shape_t& s, int n_shared = 0);
int launch_decode_one(const float* logits, const __nv_bfloat16* x, const ExpertWeights& w, const moe_shape_t& s,
                      __nv_bfloat16* out, int* ids_out, float* w_out, int* sync, void* scratch, StatusRef status,
                      cudaStream_t st, const ExpertWeights* shared = nullptr);

// router projection, join with the shared expert, and the shared expert's offsets {0, T} (moe_block.cu)
int launch_router_logits(const __nv_bfloat16* x, const __nv_bfloat16* w_router, int T, int H, int E, float* logits, int* status,
                         cudaStream_t st);
// expert-parallel sharding: the table of output rows (see moe_ep_row_table)
int launch_ep_row_table(const int* perm, const int* offsets, int k, int H, int e_begin, int e_end, float* const* owner_y, int world,
                        int tokens_per_rank, float** row_dst, cudaStream_t st, int max_rows);
int launch_combine_shared(const float* y_perm, const int* inv_perm, const float* w, const float* y_shared, const moe_shape_t& s,
                          __nv_bfloat16* out, cudaStream_t st);
int launch_shared_offsets(int* offsets2, int T, cudaStream_t st);

int sm_count();  // of the current device

// ---- per-device one-time set-up (host) ---------------------------------------------------------------
// cudaFuncSetAttribute and the SM count belong to a device, not to the process: a process that drives several GPUs
// through this library sets each kernel's attributes once on every device it calls from.
constexpr int kMaxDevices = 64;
int current_device();  // -1 if the runtime cannot tell
struct PerDeviceFlag {
  bool done[kMaxDevices] = {};
};
template <typename F>
inline bool once_per_device(PerDeviceFlag& f, F&& set) {
  const int d = current_device();
  if (d < 0 || d >= kMaxDevices) return false;
  if (!f.done[d]) {
    if (!set()) return false;
    f.done[d] = true;
  }
  return true;
}

// ---- programmatic dependent launch (host) ------------------------------------------------------
// The kernel may start while its predecessor in the stream is still running; it must execute
// griddepcontrol.wait before it reads anything the predecessor writes, and before it writes anything at all to
// global memory.  Most kernels here wait first and then release their own dependent; route_kernel, native_split_kernel
// and the expert-FFN kernels release theirs BEFORE they wait, so three or four neighbours of a chain (route, permute,
// split, expert FFN) can be resident together.  That is safe because of the rule above: whatever a kernel does before
// its wait only reads buffers that no kernel of the chain before it writes (logits, expert_offsets of a completed
// router, the weights), and every global write comes after the wait, i.e. after everything launched earlier on the
// stream has completed.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- small device helpers ---------------------------------------------------------------------
MOE_DEVINL void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
MOE_DEVINL void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

MOE_DEVINL int warp_excl_scan(int v, int lane, int* total) {
  int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += n;
  }
  *total = __shfl_sync(0xffffffffu, incl, 31);
  return incl - v;
}

}  // namespace moe
