// Read-only streaming probe: how fast one persistent CTA per SM can pull a device buffer through a shared-memory
// ring of bulk copies when nothing is done with the data.  It is the ceiling for the decode-sized expert kernel,
// whose weight stream is the same mechanism plus the tensor-core work; bench.py reports it beside the roofline.
#include "moe_sm100_primitives.cuh"

namespace moe {

namespace {
constexpr int kProbeChunk = 32 * 1024;  // bytes per bulk copy: one weight stage of the decode kernel
#ifndef MOE_PROBE_STAGES
#define MOE_PROBE_STAGES 6
#endif
constexpr int kProbeStages = MOE_PROBE_STAGES;

__global__ void __launch_bounds__(64, 1) read_probe_kernel(const uint8_t* __restrict__ src, long long n_chunks,
                                                           unsigned* __restrict__ sink, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 127) & ~uintptr_t(127));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kProbeStages * kProbeChunk);
  uint64_t* empty = full + kProbeStages;
  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int s = 0; s < kProbeStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  if (tid == 0) {  // producer
    int s = 0;
    uint32_t ph = 0;
    for (long long c = blockIdx.x; c < n_chunks; c += gridDim.x) {
      mbar_wait(&empty[s], ph ^ 1u, status);
      mbar_expect_tx(&full[s], kProbeChunk);
      bulk_g2s(smem + s * kProbeChunk, src + c * kProbeChunk, kProbeChunk, &full[s]);
      if (++s == kProbeStages) { s = 0; ph ^= 1u; }
    }
  } else if (tid == 32) {  // consumer: one word per chunk, so that the copies cannot be dropped
    int s = 0;
    uint32_t ph = 0;
    unsigned acc = 0;
    for (long long c = blockIdx.x; c < n_chunks; c += gridDim.x) {
      mbar_wait(&full[s], ph, status);
      acc ^= *reinterpret_cast<const volatile unsigned*>(smem + s * kProbeChunk);
      mbar_arrive(&empty[s]);
      if (++s == kProbeStages) { s = 0; ph ^= 1u; }
    }
    sink[blockIdx.x] = acc;
  }
}
}  // namespace

}  // namespace moe

extern "C" int moe_debug_read_probe(const void* src, size_t bytes, void* sink, size_t sink_bytes, int32_t* status_word,
                                    void* cuda_stream) {
  using namespace moe;
  if (src == nullptr || sink == nullptr || (reinterpret_cast<uintptr_t>(src) & 127u) != 0 || bytes < static_cast<size_t>(kProbeChunk) ||
      sink_bytes < static_cast<size_t>(sm_count()) * 4)
    return MOE_ERR_INVALID_ARG;
  const size_t smem = static_cast<size_t>(kProbeStages) * kProbeChunk + 2 * kProbeStages * 8 + 128;
  static PerDeviceFlag flag;
  if (!once_per_device(flag, [smem] {
        return cudaFuncSetAttribute(read_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) == cudaSuccess;
      }))
    return MOE_ERR_CUDA;
  read_probe_kernel<<<sm_count(), 64, smem, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint8_t*>(src), static_cast<long long>(bytes / kProbeChunk), static_cast<unsigned*>(sink), status_word);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
