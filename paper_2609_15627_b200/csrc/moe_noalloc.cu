// moe_expert_ffn for callers that cannot allocate device memory: the intermediate (and, for decode-sized
// batches, the E2M1 term rows of the activations) lives in a fixed array inside the library image instead of a
// caller-provided workspace.
#include "moe_common.cuh"

namespace moe {

namespace {

constexpr size_t kStaticScratchBytes = 16u << 20;  // 16 MiB

// Lives in every GPU context that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code the name of a __device__ array is only a host-side handle; the device address has to be
// asked for, per device, with that device current.
void* g_scratch_addr[kMaxDevices] = {};

int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOE_ERR_CUDA;
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return MOE_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return MOE_OK;
}

bool aligned16(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

}  // namespace moe

using namespace moe;

extern "C" {

size_t moe_expert_ffn_noalloc_max_bytes(void) { return kStaticScratchBytes; }

int moe_expert_ffn_noalloc(const void* x_perm_bf16, const int32_t* expert_offsets, const uint8_t* w13,
                           const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape,
                           float* y_perm, int32_t* status_word, void* cuda_stream) {
  if (shape == nullptr) return MOE_ERR_INVALID_ARG;
  const moe_shape_t& s = *shape;
  if (s.T < 1 || s.H < 1 || s.I < 1 || s.E < 1 || s.k < 1 || s.k > s.E) return MOE_ERR_INVALID_ARG;
  if (s.H % 128 != 0 || s.I % 128 != 0 || s.E > 1024 || s.k > 32) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(x_perm_bf16) || !aligned16(expert_offsets) || !aligned16(w13) || !aligned16(w13_scale) || !aligned16(w2) ||
      !aligned16(w2_scale) || !aligned16(y_perm))
    return MOE_ERR_INVALID_ARG;
  if (status_word != nullptr && (reinterpret_cast<uintptr_t>(status_word) & 3u) != 0) return MOE_ERR_INVALID_ARG;
  // what the chosen kernel keeps between its launches must fit the fixed array: the bf16 intermediate act[T*k, I],
  // or for the native variant the E2M1 term rows and scale bytes of both projections' inputs (4.25 (H + I) bytes per slot)
  const unsigned long long S = static_cast<unsigned long long>(s.T) * s.k;
  const unsigned long long need =
      (native_shape_ok(s, w13, w2) ? static_cast<unsigned long long>(native_scratch_bytes(s)) : S * s.I * 2ULL) + kAlign;
  if (need > kStaticScratchBytes) return MOE_ERR_WORKSPACE;
  void* scratch = nullptr;
  int rc = static_scratch(&scratch);  // first call on a device looks the address up
  if (rc != MOE_OK) return rc;
  StatusRef status;  // the caller's word, or the library's own (a second fixed device word; nothing is allocated)
  if ((rc = resolve_status(status_word, &status)) != MOE_OK) return rc;
  // Every row of act that stage 2 reads is written by stage 1 of the same call, so nothing in the array has
  // to start at zero.  Same kernels and the same kernel choice as moe_expert_ffn.
  __nv_bfloat16* act = static_cast<__nv_bfloat16*>(scratch);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const ExpertWeights w{w13, w13_scale, w2, w2_scale, false};
  if (native_shape_ok(s, w13, w2))
    return launch_expert_ffn_native(static_cast<const __nv_bfloat16*>(x_perm_bf16), expert_offsets, w, s, scratch, y_perm,
                                    status, st);
  if (status.own && cudaMemsetAsync(status.word, 0, sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
  if (umma_shape_ok(s))
    return launch_expert_ffn_umma(static_cast<const __nv_bfloat16*>(x_perm_bf16), expert_offsets, w, s, act, y_perm,
                                  status.word, st);
  return launch_expert_ffn_stream(static_cast<const __nv_bfloat16*>(x_perm_bf16), expert_offsets, w13, w13_scale, w2,
                                  w2_scale, s, act, y_perm, status.word, st);
}

}  // extern "C"
