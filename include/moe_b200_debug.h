/*
 * moe_b200_debug.h - diagnostic and measurement exports of libmoe_b200.so.
 *
 * Not part of the layer's interface (include/moe_b200.h): these calls exist for the tests and for bench.py.  None
 * has a counterpart in the paper.  Same conventions as moe_b200.h: device pointers unless stated, enqueue only,
 * moe_status_t return values, bounded device-side waits.
 */
#ifndef MOE_B200_DEBUG_H_
#define MOE_B200_DEBUG_H_

#include "moe_b200.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Measurement aid (no counterpart in the paper): one persistent CTA per SM pulls `bytes` of device memory at `src`
 * (128-byte aligned, at least 32 KB) through a shared-memory ring of 32 KB bulk copies and does nothing with them -
 * the decode-sized expert kernel's weight stream without the tensor-core work.  Timed by the caller with CUDA events
 * over a buffer larger than L2 it gives the read-only bandwidth such a stream can reach on this GPU, which bench.py
 * reports beside the roofline.  `sink` receives one word per CTA (4 * number of SMs bytes at least).  Enqueue only;
 * bounded waits as everywhere.
 */
int moe_debug_read_probe(const void* src, size_t bytes, void* sink, size_t sink_bytes, int32_t* status_word,
                         void* cuda_stream);

/* Host, pure, diagnostic.  Work split of the decode-sized expert-FFN kernel: which items (touched expert x tile of
 * 256 weight rows, in expert order) CTA `cta` of `n_ctas` takes when `n_touched` experts have rows.  out4 = first
 * and one-past-last gate/up item, first and one-past-last down item.  A down item waits, on the device, for all
 * gate/up items of its expert; the split keeps those in CTAs with a lower or equal index.  INVALID_ARG on
 * nonsense (cta outside [0, n_ctas), n_touched outside [0, 1024], H or 2I not a multiple of 256). */
int moe_debug_native_cta_share(int32_t n_ctas, int32_t cta, int32_t n_touched, int32_t H, int32_t I, int32_t* out4);

/* Diagnostic: the one-launch kernel of moe_forward for any batch it can take (up to 4 tokens, T*k <= 32), where
 * moe_forward itself would run the four calls because they are faster from 2 tokens on.  Same arguments, workspace and
 * result as moe_forward; MOE_ERR_UNSUPPORTED_SHAPE if the kernel cannot take the shape.  For the tests. */
int moe_debug_forward_one_launch(const float* logits, const void* x_bf16, const uint8_t* w13, const uint8_t* w13_scale,
                                 const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape, void* out_bf16,
                                 int32_t* topk_ids, float* topk_w, int32_t* status_word, void* ws, size_t ws_bytes,
                                 void* cuda_stream);

/*
 * moe_expert_ffn with the kernel variant chosen by the caller instead of by the shape: 0 = register-expansion
 * streaming kernel (any supported shape), 1 = bf16 tcgen05 grouped GEMM (H and I multiples of 512), 2 = block-scaled
 * FP4 tcgen05 kernel (the shapes moe_expert_ffn gives it).  Same arguments, workspace and meaning as moe_expert_ffn.
 * MOE_ERR_UNSUPPORTED_SHAPE if the variant cannot take the shape.  For tests that compare two variants on the same
 * inputs over a whole tensor, at sizes where the oracle can only be sampled.
 */
int moe_debug_expert_ffn_variant(const void* x_perm_bf16, const int32_t* expert_offsets, const uint8_t* w13,
                                 const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale,
                                 const moe_shape_t* shape, float* y_perm, int32_t* status_word, void* ws, size_t ws_bytes,
                                 void* cuda_stream, int32_t variant);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_DEBUG_H_ */
