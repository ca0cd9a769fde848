// extern "C" entry points of include/moe_b200.h: host-side argument checks, workspace carving and
// kernel selection (a pure function of the shape).  No allocation, no synchronisation, no D2H copy,
// except in moe_forward_host which is the host-buffer convenience path.
#include <string.h>

#include "moe_common.cuh"

namespace moe {

namespace {
thread_local const char* g_last_kernel = "";
thread_local uint64_t g_launches = 0;

bool aligned(const void* p, size_t a) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_shape(const moe_shape_t* s) {
  if (s == nullptr) return MOE_ERR_INVALID_ARG;
  if (s->T < 1 || s->H < 1 || s->I < 1 || s->E < 1 || s->k < 1 || s->k > s->E) return MOE_ERR_INVALID_ARG;
  if (s->H % 128 != 0 || s->I % 128 != 0 || s->E > 1024 || s->k > 32) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (static_cast<long long>(s->T) * s->k > (1LL << 30)) return MOE_ERR_UNSUPPORTED_SHAPE;
  return MOE_OK;
}

int check_ws(const void* ws, size_t ws_bytes, size_t need) {
  if (!aligned(ws, kAlign) || ws_bytes < need) return MOE_ERR_WORKSPACE;
  return MOE_OK;
}
}  // namespace

namespace {
// see StatusRef: the word used by calls whose caller passed no status word; one per device that loads the library
static __device__ int g_status_fallback;
int* g_status_fallback_addr[kMaxDevices] = {};
}  // namespace

int resolve_status(int32_t* user_word, StatusRef* out) {
  if (user_word != nullptr) {
    *out = StatusRef{user_word, false};
    return MOE_OK;
  }
  const int dev = current_device();
  if (dev < 0 || dev >= kMaxDevices) return MOE_ERR_CUDA;
  if (g_status_fallback_addr[dev] == nullptr) {
    // the name of a __device__ variable is a host-side handle: its device address is looked up per device
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_fallback) != cudaSuccess || p == nullptr) return MOE_ERR_CUDA;
    g_status_fallback_addr[dev] = static_cast<int*>(p);
  }
  *out = StatusRef{g_status_fallback_addr[dev], true};
  return MOE_OK;
}

// kernels that cannot clear the library's own status word themselves: a memset node before them
static int clear_own_status(const StatusRef& s, cudaStream_t st) {
  if (s.own && cudaMemsetAsync(s.word, 0, sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

void note_kernel(const char* name, int launches) {
  g_last_kernel = name;
  g_launches += static_cast<uint64_t>(launches);
}

int current_device() {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

int sm_count() {
  static int n[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0 || dev >= kMaxDevices) return 148;
  if (n[dev] == 0 && (cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n[dev] <= 0))
    n[dev] = 148;
  return n[dev];
}

}  // namespace moe

using namespace moe;

extern "C" {

size_t moe_workspace_bytes(const moe_shape_t* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  return ws_layout(*shape).total;
}

const char* moe_status_string(int status) {
  switch (status) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case MOE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MOE_ERR_CUDA: return "CUDA runtime or launch error";
    case MOE_ERR_TIMEOUT: return "device-side bounded wait ran out";
    default: return "unknown status";
  }
}

const char* moe_last_kernel_name(void) { return g_last_kernel; }

uint64_t moe_launch_count(void) { return g_launches; }

int moe_route(const float* logits, int32_t T, int32_t E, int32_t k, int32_t* topk_ids, float* topk_w,
              int32_t* expert_offsets, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (T < 1 || E < 1 || k < 1 || k > E) return MOE_ERR_INVALID_ARG;
  if (E > 1024 || k > 32 || static_cast<long long>(T) * k > (1LL << 30)) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (!aligned(logits, 16) || !aligned(topk_ids, 16) || !aligned(topk_w, 16) || !aligned(expert_offsets, 16))
    return MOE_ERR_INVALID_ARG;
  // route uses only the counter block at the start of the workspace
  const size_t need = align_up((static_cast<size_t>(E) + 8) * 4, kAlign);
  if (check_ws(ws, ws_bytes, need) != MOE_OK) return MOE_ERR_WORKSPACE;
  int* counters = static_cast<int*>(ws);
  return launch_route(logits, T, E, k, topk_ids, topk_w, expert_offsets, counters, static_cast<cudaStream_t>(cuda_stream));
}

int moe_permute(const void* x_bf16, const int32_t* topk_ids, const int32_t* expert_offsets, const moe_shape_t* shape,
                void* x_perm_bf16, int32_t* perm, int32_t* inv_perm, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(x_bf16, 16) || !aligned(topk_ids, 16) || !aligned(expert_offsets, 16) || !aligned(x_perm_bf16, 16) ||
      !aligned(perm, 16) || !aligned(inv_perm, 16))
    return MOE_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*shape);
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  int* block_counts = reinterpret_cast<int*>(static_cast<char*>(ws) + L.permute_off);
  return launch_permute(static_cast<const __nv_bfloat16*>(x_bf16), topk_ids, expert_offsets, *shape,
                        static_cast<__nv_bfloat16*>(x_perm_bf16), perm, inv_perm, block_counts,
                        static_cast<cudaStream_t>(cuda_stream));
}

namespace {
int expert_ffn_impl(const void* x_perm_bf16, const int32_t* expert_offsets, const ExpertWeights& w, const moe_shape_t* shape,
                    float* y_perm, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream,
                    float* const* row_dst = nullptr, const moe_shape_t* choice = nullptr) {
  // `choice`: the shape that picks the kernel where it is not `shape` itself - a rank of an expert-parallel job runs the
  // kernel the unsharded layer would run, so that the sharded result has the same bits
  if (choice == nullptr) choice = shape;
  if (!aligned(x_perm_bf16, 16) || !aligned(expert_offsets, 16) || !aligned(w.w13, 16) || !aligned(w.s13, 16) ||
      !aligned(w.w2, 16) || !aligned(w.s2, 16) || (row_dst == nullptr ? !aligned(y_perm, 16) : !aligned(row_dst, 8)))
    return MOE_ERR_INVALID_ARG;  // (with a table of output rows there is no y_perm)
  if (status_word != nullptr && !aligned(status_word, 4)) return MOE_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*choice);  // (the scratch of the kernel that `choice` picks, same row count)
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  __nv_bfloat16* act = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + L.act_off);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const __nv_bfloat16* xp = static_cast<const __nv_bfloat16*>(x_perm_bf16);
  // kernel choice is a pure function of the shape (and of the alignment the tensor maps need): native block-scaled
  // FP4 MMA for decode-sized batches, bf16 grouped GEMM for prefill-sized batches, the register-expansion streaming
  // kernel for every other shape.  The streaming kernel reads whole rows, so with the tile-contiguous weight layout
  // (which only shapes the first two kernels take can have) the grouped GEMM also takes what is left.
  StatusRef status;
  int rc = resolve_status(status_word, &status);
  if (rc != MOE_OK) return rc;
  if (native_shape_ok(*choice, w.w13, w.w2))
    return launch_expert_ffn_native(xp, expert_offsets, w, *shape, act, y_perm, status, st, row_dst);
  if ((rc = clear_own_status(status, st)) != MOE_OK) return rc;
  if (umma_shape_ok(*choice) || w.blocked)
    return launch_expert_ffn_umma(xp, expert_offsets, w, *shape, act, y_perm, status.word, st, row_dst);
  return launch_expert_ffn_stream(xp, expert_offsets, w.w13, w.s13, w.w2, w.s2, *shape, act, y_perm, status.word, st, row_dst);
}

// the four tensors inside a buffer written by moe_prepack
ExpertWeights packed_view(const void* packed, const moe_shape_t& s) {
  const PackedLayout L = packed_layout(s);
  const uint8_t* b = static_cast<const uint8_t*>(packed);
  return ExpertWeights{b + L.w13, b + L.s13, b + L.w2, b + L.s2, blocked_shape(s)};
}
}  // namespace

int moe_expert_ffn(const void* x_perm_bf16, const int32_t* expert_offsets, const uint8_t* w13, const uint8_t* w13_scale,
                   const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape, float* y_perm,
                   int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  return expert_ffn_impl(x_perm_bf16, expert_offsets, ExpertWeights{w13, w13_scale, w2, w2_scale, false}, shape, y_perm,
                         status_word, ws, ws_bytes, cuda_stream);
}

size_t moe_prepack_bytes(const moe_shape_t* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  return packed_layout(*shape).total;
}

int moe_prepack(const uint8_t* w13, const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale,
                const moe_shape_t* shape, void* packed_out, size_t packed_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(w13, 16) || !aligned(w13_scale, 16) || !aligned(w2, 16) || !aligned(w2_scale, 16)) return MOE_ERR_INVALID_ARG;
  if (!aligned(packed_out, kAlign) || packed_bytes < packed_layout(*shape).total) return MOE_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // load check of the scale bytes (once per model load, so a round trip to the host is affordable): the kernels
  // take bytes 0..128 only, and a larger one would give silently unspecified values on the hot path
  StatusRef counter;  // the library's own device word doubles as the counter of this one-time check
  if (resolve_status(nullptr, &counter) != MOE_OK) return MOE_ERR_CUDA;
  const size_t n = static_cast<size_t>(shape->E) * shape->H * shape->I;
  const uint8_t* tensors[2] = {w13_scale, w2_scale};
  const size_t sizes[2] = {n / 16, n / 32};
  for (int i = 0; i < 2; ++i) {
    int bad = 0;
    if (launch_validate_scales(tensors[i], sizes[i], counter.word, st) != MOE_OK ||
        cudaMemcpyAsync(&bad, counter.word, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
      return MOE_ERR_CUDA;
    if (bad != 0) {
      cudaMemsetAsync(counter.word, 0, sizeof(int), st);
      return MOE_ERR_INVALID_ARG;
    }
  }
  return launch_prepack(w13, w13_scale, w2, w2_scale, *shape, static_cast<uint8_t*>(packed_out), st);
}

int moe_expert_ffn_packed(const void* x_perm_bf16, const int32_t* expert_offsets, const void* packed, const moe_shape_t* shape,
                          float* y_perm, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(packed, kAlign)) return MOE_ERR_INVALID_ARG;
  return expert_ffn_impl(x_perm_bf16, expert_offsets, packed_view(packed, *shape), shape, y_perm, status_word, ws, ws_bytes,
                         cuda_stream);
}

int moe_combine(const float* y_perm, const int32_t* inv_perm, const float* topk_w, const moe_shape_t* shape,
                void* out_bf16, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(y_perm, 16) || !aligned(inv_perm, 16) || !aligned(topk_w, 16) || !aligned(out_bf16, 16))
    return MOE_ERR_INVALID_ARG;
  return launch_combine(y_perm, inv_perm, topk_w, *shape, static_cast<__nv_bfloat16*>(out_bf16),
                        static_cast<cudaStream_t>(cuda_stream));
}

// ---- router projection, shared expert, join: the whole FFN block ---------------------------------------------
int moe_router_logits(const void* x_bf16, const void* w_router_bf16, int32_t T, int32_t H, int32_t E, float* logits,
                      int32_t* status_word, void* cuda_stream) {
  if (T < 1 || H < 1 || E < 1) return MOE_ERR_INVALID_ARG;
  if (H % 128 != 0 || E > 1024) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (!aligned(x_bf16, 16) || !aligned(w_router_bf16, 16) || !aligned(logits, 16) ||
      (status_word != nullptr && !aligned(status_word, 4)))
    return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  StatusRef status;
  int rc = resolve_status(status_word, &status);
  if (rc != MOE_OK) return rc;
  if ((rc = clear_own_status(status, st)) != MOE_OK) return rc;
  return launch_router_logits(static_cast<const __nv_bfloat16*>(x_bf16), static_cast<const __nv_bfloat16*>(w_router_bf16), T, H, E,
                              logits, status.word, st);
}

int moe_combine_shared(const float* y_perm, const int32_t* inv_perm, const float* topk_w, const float* y_shared,
                       const moe_shape_t* shape, void* out_bf16, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(y_perm, 16) || !aligned(inv_perm, 16) || !aligned(topk_w, 16) || !aligned(y_shared, 16) || !aligned(out_bf16, 16))
    return MOE_ERR_INVALID_ARG;
  return launch_combine_shared(y_perm, inv_perm, topk_w, y_shared, *shape, static_cast<__nv_bfloat16*>(out_bf16),
                               static_cast<cudaStream_t>(cuda_stream));
}

namespace {
// ws of moe_ffn_block = [ logits | ids | w | offsets | shared offsets | x_perm | perm | inv_perm | y_perm | y_shared |
//                         the expert-FFN calls' workspace (the routed call's and the shared call's, used one after the other) ]
struct BlockLayout {
  size_t logits, ids, w, offsets, offsets2, x_perm, perm, inv_perm, y_perm, y_shared, inner, inner_bytes, one_sync, one_scratch, total;
};
moe_shape_t shared_shape(const moe_shape_t& s) { return moe_shape_t{s.T, s.H, s.I, 1, 1}; }
BlockLayout block_layout(const moe_shape_t& s) {
  BlockLayout L;
  const size_t S = static_cast<size_t>(s.T) * s.k;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align_up(bytes, kAlign);
    return o;
  };
  L.logits = take(static_cast<size_t>(s.T) * s.E * 4);
  L.ids = take(S * 4);
  L.w = take(S * 4);
  L.offsets = take((static_cast<size_t>(s.E) + 1) * 4);
  L.offsets2 = take(16);
  L.x_perm = take(S * s.H * 2);
  L.perm = take(S * 4);
  L.inv_perm = take(S * 4);
  L.y_perm = take(S * s.H * 4);
  L.y_shared = take(static_cast<size_t>(s.T) * s.H * 4);
  L.inner = off;
  const size_t a = ws_layout(s).total, b = ws_layout(shared_shape(s)).total;
  L.inner_bytes = a > b ? a : b;
  off += L.inner_bytes;
  // one token: the counter block and the scratch of the one-launch kernel with the shared expert as an extra slot
  // (whether that kernel applies also depends on the weights' alignment; the size allows for it whenever the shape does)
  const void* al = reinterpret_cast<const void*>(uintptr_t(256));
  L.one_sync = take(kForwardSyncBytes);
  L.one_scratch = take(decode_one_ok(s, al, al, 1) ? decode_one_scratch_bytes(s, 1) : 0);
  L.total = off;
  return L;
}
}  // namespace

// ---- expert-parallel sharding ------------------------------------------------------------------------
namespace {
int check_ep(const moe_shape_t& s, int e_begin, int e_end, int world) {
  if (world < 1 || e_begin < 0 || e_end <= e_begin || e_end > s.E) return MOE_ERR_INVALID_ARG;
  if (e_begin % 4 != 0) return MOE_ERR_INVALID_ARG;  // the shifted offsets array keeps its 16-byte alignment
  return MOE_OK;
}
}  // namespace

int moe_ep_permute(const void* x_bf16, const int32_t* topk_ids, const int32_t* expert_offsets, const moe_shape_t* shape, int32_t e_begin,
                   int32_t e_end, void* x_perm_bf16, int32_t* perm, int32_t* inv_perm, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if ((rc = check_ep(*shape, e_begin, e_end, 1)) != MOE_OK) return rc;
  if (!aligned(x_bf16, 16) || !aligned(topk_ids, 16) || !aligned(expert_offsets, 16) || !aligned(x_perm_bf16, 16) ||
      !aligned(perm, 16) || !aligned(inv_perm, 16))
    return MOE_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*shape);
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  int* block_counts = reinterpret_cast<int*>(static_cast<char*>(ws) + L.permute_off);
  return launch_permute(static_cast<const __nv_bfloat16*>(x_bf16), topk_ids, expert_offsets, *shape,
                        static_cast<__nv_bfloat16*>(x_perm_bf16), perm, inv_perm, block_counts, static_cast<cudaStream_t>(cuda_stream),
                        expert_offsets + e_begin, expert_offsets + e_end);
}

int moe_ep_row_table(const int32_t* perm, const int32_t* expert_offsets, const moe_shape_t* shape, int32_t e_begin, int32_t e_end,
                     float* const* owner_y, int32_t world, float** row_dst, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if ((rc = check_ep(*shape, e_begin, e_end, world)) != MOE_OK) return rc;
  if (perm == nullptr || expert_offsets == nullptr || owner_y == nullptr || row_dst == nullptr) return MOE_ERR_INVALID_ARG;
  const int tpr = (shape->T + world - 1) / world;
  return launch_ep_row_table(perm, expert_offsets, shape->k, shape->H, e_begin, e_end, owner_y, world, tpr, row_dst,
                             static_cast<cudaStream_t>(cuda_stream), shape->T * shape->k);
}

int moe_ep_expert_ffn(const void* x_perm_bf16, const int32_t* expert_offsets, const uint8_t* w13_local, const uint8_t* w13_scale_local,
                      const uint8_t* w2_local, const uint8_t* w2_scale_local, const moe_shape_t* shape, int32_t e_begin, int32_t e_end,
                      float* const* row_dst, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if ((rc = check_ep(*shape, e_begin, e_end, 1)) != MOE_OK) return rc;
  if (row_dst == nullptr || expert_offsets == nullptr) return MOE_ERR_INVALID_ARG;
  // the kernels see this rank's experts only: their rows are the range [offsets[e_begin], offsets[e_end]) of the sorted
  // order, and the shifted offsets array describes exactly that; x_perm and the table are indexed by sorted row as ever
  moe_shape_t local = *shape;
  local.E = e_end - e_begin;  // (k stays: it only sizes buffers and tensor maps, T * k rows)
  return expert_ffn_impl(x_perm_bf16, expert_offsets + e_begin, ExpertWeights{w13_local, w13_scale_local, w2_local, w2_scale_local, false},
                         &local, nullptr, status_word, ws, ws_bytes, cuda_stream, row_dst, shape);
}

size_t moe_expert_ffn_q_workspace_bytes(const moe_shape_t* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  return native_q_scratch_bytes(*shape) + kAlign;
}

int moe_expert_ffn_q(const void* x_perm_bf16, const int32_t* expert_offsets, const uint8_t* w13, const uint8_t* w13_scale,
                     const uint8_t* w2, const uint8_t* w2_scale, const void* packed, const moe_shape_t* shape, float* y_perm,
                     int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  const bool raw = w13 != nullptr || w13_scale != nullptr || w2 != nullptr || w2_scale != nullptr;
  if (raw == (packed != nullptr)) return MOE_ERR_INVALID_ARG;  // exactly one form of the weights
  if (packed != nullptr && !aligned(packed, kAlign)) return MOE_ERR_INVALID_ARG;
  const ExpertWeights w = packed != nullptr ? packed_view(packed, *shape) : ExpertWeights{w13, w13_scale, w2, w2_scale, false};
  if (w.w13 == nullptr || w.s13 == nullptr || w.w2 == nullptr || w.s2 == nullptr || x_perm_bf16 == nullptr ||
      expert_offsets == nullptr || y_perm == nullptr)
    return MOE_ERR_INVALID_ARG;
  if (!aligned(x_perm_bf16, 16) || !aligned(expert_offsets, 16) || !aligned(w.w13, 16) || !aligned(w.s13, 16) ||
      !aligned(w.w2, 16) || !aligned(w.s2, 16) || !aligned(y_perm, 16))
    return MOE_ERR_INVALID_ARG;
  if (status_word != nullptr && !aligned(status_word, 4)) return MOE_ERR_INVALID_ARG;
  if (!native_q_shape_ok(*shape, w.w13, w.w2)) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (check_ws(ws, ws_bytes, native_q_scratch_bytes(*shape)) != MOE_OK) return MOE_ERR_WORKSPACE;
  StatusRef status;
  if ((rc = resolve_status(status_word, &status)) != MOE_OK) return rc;
  return launch_expert_ffn_native_q(static_cast<const __nv_bfloat16*>(x_perm_bf16), expert_offsets, w, *shape, ws, y_perm, status,
                                    static_cast<cudaStream_t>(cuda_stream));
}

size_t moe_ffn_block_workspace_bytes(const moe_shape_t* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  return block_layout(*shape).total;
}

int moe_ffn_block(const void* x_bf16, const void* w_router_bf16, const uint8_t* w13, const uint8_t* w13_scale, const uint8_t* w2,
                  const uint8_t* w2_scale, const uint8_t* shared_w13, const uint8_t* shared_w13_scale, const uint8_t* shared_w2,
                  const uint8_t* shared_w2_scale, const moe_shape_t* shape, void* out_bf16, int32_t* topk_ids, float* topk_w,
                  int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(x_bf16, 16) || !aligned(w_router_bf16, 16) || !aligned(out_bf16, 16) || !aligned(shared_w13, 16) ||
      !aligned(shared_w13_scale, 16) || !aligned(shared_w2, 16) || !aligned(shared_w2_scale, 16) ||
      (topk_ids != nullptr && !aligned(topk_ids, 16)) || (topk_w != nullptr && !aligned(topk_w, 16)))
    return MOE_ERR_INVALID_ARG;
  const moe_shape_t& s = *shape;
  const BlockLayout L = block_layout(s);
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* d_logits = reinterpret_cast<float*>(base + L.logits);
  int32_t* d_ids = topk_ids != nullptr ? topk_ids : reinterpret_cast<int32_t*>(base + L.ids);
  float* d_w = topk_w != nullptr ? topk_w : reinterpret_cast<float*>(base + L.w);
  int32_t* d_off = reinterpret_cast<int32_t*>(base + L.offsets);
  int32_t* d_off2 = reinterpret_cast<int32_t*>(base + L.offsets2);
  void* d_xp = base + L.x_perm;
  int32_t* d_perm = reinterpret_cast<int32_t*>(base + L.perm);
  int32_t* d_inv = reinterpret_cast<int32_t*>(base + L.inv_perm);
  float* d_y = reinterpret_cast<float*>(base + L.y_perm);
  float* d_ys = reinterpret_cast<float*>(base + L.y_shared);
  void* inner = base + L.inner;
  const moe_shape_t sh1 = shared_shape(s);
  // router scores -> Top-k -> route production -> routed experts; the shared expert on every token (its sorted rows are
  // the token rows themselves); the join
  if (decode_one_ok(s, w13, w2, 1) && aligned(shared_w13, 16) && aligned(shared_w2, 16) && s.H % 512 == 0 && s.I % 512 == 0) {
    // One token: the router projection, then ONE launch for everything else - the shared expert is one more slot of the
    // one-token kernel (its weights depend on no routing, so its stream starts first), added with weight 1 after the
    // routed slots' recurrence.  The kernel needs its counter block clear; this call owns the block.
    if (cudaMemsetAsync(base + L.one_sync, 0, kForwardSyncBytes, st) != cudaSuccess) return MOE_ERR_CUDA;
    if ((rc = moe_router_logits(x_bf16, w_router_bf16, s.T, s.H, s.E, d_logits, status_word, st)) != MOE_OK) return rc;
    StatusRef status;
    if ((rc = resolve_status(status_word, &status)) != MOE_OK) return rc;
    const ExpertWeights shared{shared_w13, shared_w13_scale, shared_w2, shared_w2_scale, false};
    return launch_decode_one(d_logits, static_cast<const __nv_bfloat16*>(x_bf16), ExpertWeights{w13, w13_scale, w2, w2_scale, false}, s,
                             static_cast<__nv_bfloat16*>(out_bf16), topk_ids, topk_w, reinterpret_cast<int*>(base + L.one_sync),
                             base + L.one_scratch, status, st, &shared);
  }
  if ((rc = moe_router_logits(x_bf16, w_router_bf16, s.T, s.H, s.E, d_logits, status_word, st)) != MOE_OK) return rc;
  if ((rc = launch_shared_offsets(d_off2, s.T, st)) != MOE_OK) return rc;
  if ((rc = moe_route(d_logits, s.T, s.E, s.k, d_ids, d_w, d_off, inner, L.inner_bytes, st)) != MOE_OK) return rc;
  if ((rc = moe_permute(x_bf16, d_ids, d_off, shape, d_xp, d_perm, d_inv, inner, L.inner_bytes, st)) != MOE_OK) return rc;
  if ((rc = moe_expert_ffn(d_xp, d_off, w13, w13_scale, w2, w2_scale, shape, d_y, status_word, inner, L.inner_bytes, st)) != MOE_OK)
    return rc;
  if ((rc = moe_expert_ffn(x_bf16, d_off2, shared_w13, shared_w13_scale, shared_w2, shared_w2_scale, &sh1, d_ys, status_word, inner,
                           L.inner_bytes, st)) != MOE_OK)
    return rc;
  return moe_combine_shared(d_y, d_inv, d_w, d_ys, shape, out_bf16, st);
}

int moe_validate_scales(const uint8_t* scales, size_t n_bytes, int32_t* bad_count, void* cuda_stream) {
  if (scales == nullptr || n_bytes == 0 || !aligned(bad_count, 4)) return MOE_ERR_INVALID_ARG;
  return launch_validate_scales(scales, n_bytes, bad_count, static_cast<cudaStream_t>(cuda_stream));
}

// ---- whole layer, device buffers -------------------------------------------------------------------
namespace {
// ws of moe_forward = [ sync block | one-launch scratch, or the buffers between the four calls and their workspace ]
struct ForwardLayout {
  size_t ids, w, offsets, x_perm, perm, inv_perm, y_perm, inner, total;
};
ForwardLayout forward_layout(const moe_shape_t& s) {
  ForwardLayout L;
  const size_t S = static_cast<size_t>(s.T) * s.k;
  size_t off = kForwardSyncBytes;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align_up(bytes, kAlign);
    return o;
  };
  L.ids = take(S * 4);
  L.w = take(S * 4);
  L.offsets = take((static_cast<size_t>(s.E) + 1) * 4);
  L.x_perm = take(S * s.H * 2);
  L.perm = take(S * 4);
  L.inv_perm = take(S * 4);
  L.y_perm = take(S * s.H * 4);
  L.inner = off;
  off += ws_layout(s).total;
  // whether the one-launch kernel applies also depends on the weights' alignment; the size allows for it whenever
  // the shape does
  const void* al = reinterpret_cast<const void*>(uintptr_t(256));
  const size_t fused = forward_fused_ok(s, al, al) ? kForwardSyncBytes + forward_fused_scratch_bytes(s) : 0;
  const size_t one = decode_one_ok(s, al, al) ? kForwardSyncBytes + decode_one_scratch_bytes(s) : 0;
  L.total = off > fused ? off : fused;
  L.total = L.total > one ? L.total : one;
  return L;
}
}  // namespace

size_t moe_forward_workspace_bytes(const moe_shape_t* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  return forward_layout(*shape).total;
}

size_t moe_forward_sync_bytes(void) { return kForwardSyncBytes; }

namespace {
int forward_impl(const float* logits, const void* x_bf16, const ExpertWeights& w, const moe_shape_t* shape, void* out_bf16,
                 int32_t* topk_ids, float* topk_w, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc;
  if (!aligned(logits, 16) || !aligned(x_bf16, 16) || !aligned(w.w13, 16) || !aligned(w.s13, 16) || !aligned(w.w2, 16) ||
      !aligned(w.s2, 16) || !aligned(out_bf16, 16))
    return MOE_ERR_INVALID_ARG;
  if ((topk_ids != nullptr && !aligned(topk_ids, 16)) || (topk_w != nullptr && !aligned(topk_w, 16)) ||
      (status_word != nullptr && !aligned(status_word, 4)))
    return MOE_ERR_INVALID_ARG;
  const ForwardLayout L = forward_layout(*shape);
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (decode_one_ok(*shape, w.w13, w.w2)) {
    StatusRef status;
    if ((rc = resolve_status(status_word, &status)) != MOE_OK) return rc;
    return launch_decode_one(logits, static_cast<const __nv_bfloat16*>(x_bf16), w, *shape, static_cast<__nv_bfloat16*>(out_bf16),
                             topk_ids, topk_w, reinterpret_cast<int*>(base), base + kForwardSyncBytes, status, st);
  }
  if (forward_fused_ok(*shape, w.w13, w.w2) && forward_fused_preferred(*shape)) {
    StatusRef status;
    if ((rc = resolve_status(status_word, &status)) != MOE_OK) return rc;
    return launch_forward_fused(logits, static_cast<const __nv_bfloat16*>(x_bf16), w, *shape,
                                static_cast<__nv_bfloat16*>(out_bf16), topk_ids, topk_w, reinterpret_cast<int*>(base),
                                base + kForwardSyncBytes, status, st);
  }
  int32_t* d_ids = topk_ids != nullptr ? topk_ids : reinterpret_cast<int32_t*>(base + L.ids);
  float* d_w = topk_w != nullptr ? topk_w : reinterpret_cast<float*>(base + L.w);
  int32_t* d_off = reinterpret_cast<int32_t*>(base + L.offsets);
  void* d_xp = base + L.x_perm;
  int32_t* d_perm = reinterpret_cast<int32_t*>(base + L.perm);
  int32_t* d_inv = reinterpret_cast<int32_t*>(base + L.inv_perm);
  float* d_y = reinterpret_cast<float*>(base + L.y_perm);
  void* inner = base + L.inner;
  const size_t inner_bytes = ws_bytes - L.inner;
  const moe_shape_t& s = *shape;
  if ((rc = moe_route(logits, s.T, s.E, s.k, d_ids, d_w, d_off, inner, inner_bytes, st)) != MOE_OK) return rc;
  if ((rc = moe_permute(x_bf16, d_ids, d_off, shape, d_xp, d_perm, d_inv, inner, inner_bytes, st)) != MOE_OK) return rc;
  if ((rc = expert_ffn_impl(d_xp, d_off, w, shape, d_y, status_word, inner, inner_bytes, st)) != MOE_OK) return rc;
  return moe_combine(d_y, d_inv, d_w, shape, out_bf16, st);
}
}  // namespace

int moe_forward(const float* logits, const void* x_bf16, const uint8_t* w13, const uint8_t* w13_scale, const uint8_t* w2,
                const uint8_t* w2_scale, const moe_shape_t* shape, void* out_bf16, int32_t* topk_ids, float* topk_w,
                int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  return forward_impl(logits, x_bf16, ExpertWeights{w13, w13_scale, w2, w2_scale, false}, shape, out_bf16, topk_ids, topk_w,
                      status_word, ws, ws_bytes, cuda_stream);
}

int moe_debug_forward_one_launch(const float* logits, const void* x_bf16, const uint8_t* w13, const uint8_t* w13_scale,
                                 const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape, void* out_bf16,
                                 int32_t* topk_ids, float* topk_w, int32_t* status_word, void* ws, size_t ws_bytes,
                                 void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(logits, 16) || !aligned(x_bf16, 16) || !aligned(w13, 16) || !aligned(w13_scale, 16) || !aligned(w2, 16) ||
      !aligned(w2_scale, 16) || !aligned(out_bf16, 16) || (topk_ids != nullptr && !aligned(topk_ids, 16)) ||
      (topk_w != nullptr && !aligned(topk_w, 16)) || (status_word != nullptr && !aligned(status_word, 4)))
    return MOE_ERR_INVALID_ARG;
  if (!forward_fused_ok(*shape, w13, w2)) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (check_ws(ws, ws_bytes, forward_layout(*shape).total) != MOE_OK) return MOE_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  StatusRef status;
  const int rs = resolve_status(status_word, &status);
  if (rs != MOE_OK) return rs;
  return launch_forward_fused(logits, static_cast<const __nv_bfloat16*>(x_bf16), ExpertWeights{w13, w13_scale, w2, w2_scale, false},
                              *shape, static_cast<__nv_bfloat16*>(out_bf16), topk_ids, topk_w, reinterpret_cast<int*>(base),
                              base + kForwardSyncBytes, status, static_cast<cudaStream_t>(cuda_stream));
}

int moe_debug_expert_ffn_variant(const void* x_perm_bf16, const int32_t* expert_offsets, const uint8_t* w13,
                                 const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape,
                                 float* y_perm, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream,
                                 int32_t variant) {
  int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(x_perm_bf16, 16) || !aligned(expert_offsets, 16) || !aligned(w13, 16) || !aligned(w13_scale, 16) ||
      !aligned(w2, 16) || !aligned(w2_scale, 16) || !aligned(y_perm, 16) || variant < 0 || variant > 2 ||
      (status_word != nullptr && !aligned(status_word, 4)))
    return MOE_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*shape);
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  __nv_bfloat16* act = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) + L.act_off);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const __nv_bfloat16* xp = static_cast<const __nv_bfloat16*>(x_perm_bf16);
  const ExpertWeights w{w13, w13_scale, w2, w2_scale, false};
  StatusRef status;
  if ((rc = resolve_status(status_word, &status)) != MOE_OK) return rc;
  if (variant == 2) {
    if (!native_shape_ok(*shape, w13, w2)) return MOE_ERR_UNSUPPORTED_SHAPE;
    return launch_expert_ffn_native(xp, expert_offsets, w, *shape, act, y_perm, status, st);
  }
  if ((rc = clear_own_status(status, st)) != MOE_OK) return rc;
  if (variant == 1) {
    if (!blocked_shape(*shape) || !umma_shape_ok(moe_shape_t{1 << 20, shape->H, shape->I, shape->E, 1})) return MOE_ERR_UNSUPPORTED_SHAPE;
    return launch_expert_ffn_umma(xp, expert_offsets, w, *shape, act, y_perm, status.word, st);
  }
  return launch_expert_ffn_stream(xp, expert_offsets, w13, w13_scale, w2, w2_scale, *shape, act, y_perm, status.word, st);
}

int moe_forward_packed(const float* logits, const void* x_bf16, const void* packed, const moe_shape_t* shape, void* out_bf16,
                       int32_t* topk_ids, float* topk_w, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(packed, kAlign)) return MOE_ERR_INVALID_ARG;
  return forward_impl(logits, x_bf16, packed_view(packed, *shape), shape, out_bf16, topk_ids, topk_w, status_word, ws, ws_bytes,
                      cuda_stream);
}

// ---- host-buffer path ---------------------------------------------------------------------------
namespace {
struct HostLayout {
  size_t logits, x, out, inner, total;
};
HostLayout host_layout(const moe_shape_t& s) {
  HostLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align_up(bytes, kAlign);
    return o;
  };
  // (the logits sit right in front of moe_forward's workspace, whose first bytes are its counter block: small logits
  // and the block's zeros arrive in one copy)
  L.x = take(static_cast<size_t>(s.T) * s.H * 2);
  L.out = take(static_cast<size_t>(s.T) * s.H * 2);
  L.logits = take(static_cast<size_t>(s.T) * s.E * 4);
  L.inner = off;
  off += forward_layout(s).total;
  L.total = off;
  return L;
}
}  // namespace

size_t moe_forward_host_workspace_bytes(const moe_shape_t* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  return host_layout(*shape).total;
}

namespace {
constexpr size_t kStageLogitsBytes = 64 * 1024;  // logits up to this size travel together with the counter block's zeros
// [kStageLogitsBytes of logits][kForwardSyncBytes of zeros], page-locked, one per host thread (never freed)
unsigned char* logits_staging() {
  thread_local unsigned char* buf = nullptr;
  thread_local bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    if (cudaHostAlloc(&p, kStageLogitsBytes + kForwardSyncBytes, cudaHostAllocDefault) == cudaSuccess) {
      buf = static_cast<unsigned char*>(p);
      memset(buf, 0, kStageLogitsBytes + kForwardSyncBytes);
    } else {
      cudaGetLastError();
    }
  }
  return buf;
}
constexpr size_t kDirectOutBytes = 64 * 1024;  // outputs up to this size are written to pinned host memory by the kernel
int forward_host_impl(const float* logits_host, const void* x_host_bf16, const ExpertWeights& w, const moe_shape_t* shape,
                      void* out_host_bf16, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  int rc;
  if (logits_host == nullptr || x_host_bf16 == nullptr || out_host_bf16 == nullptr) return MOE_ERR_INVALID_ARG;
  const HostLayout L = host_layout(*shape);
  if (check_ws(ws, ws_bytes, L.total) != MOE_OK) return MOE_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const moe_shape_t& s = *shape;
  float* d_logits = reinterpret_cast<float*>(base + L.logits);
  void* d_x = base + L.x;
  void* d_out = base + L.out;
  // A small output goes straight to the caller's buffer where the device can address it (pinned host memory under
  // unified addressing): the last kernel's stores cross the bus instead of a copy operation enqueued after it.
  bool direct = false;
  const size_t out_bytes = static_cast<size_t>(s.T) * s.H * 2;
  if (out_bytes <= kDirectOutBytes) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, out_host_bf16) == cudaSuccess && at.type == cudaMemoryTypeHost &&
        at.devicePointer != nullptr && aligned(at.devicePointer, 16)) {
      d_out = at.devicePointer;
      direct = true;
    } else {
      cudaGetLastError();  // pageable memory: not an error of this call
    }
  }
  // Likewise a single token row is read where it lies: the few CTAs that split it fetch 512 bytes each across the bus,
  // which costs the kernel less than a copy operation in front of it costs the call.
  bool x_direct = false;
  if (s.T == 1 && decode_one_ok(s, w.w13, w.w2)) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, x_host_bf16) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer != nullptr &&
        aligned(at.devicePointer, 16)) {
      d_x = at.devicePointer;
      x_direct = true;
    } else {
      cudaGetLastError();
    }
  }
  // This call owns its workspace's contents: it clears the counter block of moe_forward itself.  Small logits go through
  // a page-locked staging buffer of this thread that ends in zeros, so that one copy brings both (the call waits for the
  // stream before it returns, so the buffer is free again by then).
  const size_t lg_bytes = static_cast<size_t>(s.T) * s.E * 4, lg_span = L.inner - L.logits;
  unsigned char* stage = lg_span <= kStageLogitsBytes ? logits_staging() : nullptr;
  if (stage != nullptr) {
    memcpy(stage, logits_host, lg_bytes);
    memset(stage + lg_bytes, 0, lg_span - lg_bytes + kForwardSyncBytes);  // (an earlier, larger batch may have left logits there)
    if (cudaMemcpyAsync(d_logits, stage, lg_span + kForwardSyncBytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return MOE_ERR_CUDA;
  } else if (cudaMemsetAsync(base + L.inner, 0, kForwardSyncBytes, st) != cudaSuccess ||
             cudaMemcpyAsync(d_logits, logits_host, lg_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    return MOE_ERR_CUDA;
  }
  if ((!x_direct && cudaMemcpyAsync(d_x, x_host_bf16, static_cast<size_t>(s.T) * s.H * 2, cudaMemcpyHostToDevice, st) != cudaSuccess))
    return MOE_ERR_CUDA;
  if ((rc = forward_impl(d_logits, d_x, w, shape, d_out, nullptr, nullptr, status_word, base + L.inner, ws_bytes - L.inner,
                         st)) != MOE_OK)
    return rc;
  if (!direct && cudaMemcpyAsync(out_host_bf16, d_out, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}
}  // namespace

int moe_forward_host(const float* logits_host, const void* x_host_bf16, const uint8_t* w13, const uint8_t* w13_scale,
                     const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape, void* out_host_bf16,
                     int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  return forward_host_impl(logits_host, x_host_bf16, ExpertWeights{w13, w13_scale, w2, w2_scale, false}, shape, out_host_bf16,
                           status_word, ws, ws_bytes, cuda_stream);
}

int moe_forward_host_packed(const float* logits_host, const void* x_host_bf16, const void* packed, const moe_shape_t* shape,
                            void* out_host_bf16, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream) {
  const int rc = check_shape(shape);
  if (rc != MOE_OK) return rc;
  if (!aligned(packed, kAlign)) return MOE_ERR_INVALID_ARG;
  return forward_host_impl(logits_host, x_host_bf16, packed_view(packed, *shape), shape, out_host_bf16, status_word, ws,
                           ws_bytes, cuda_stream);
}

}  // extern "C"
