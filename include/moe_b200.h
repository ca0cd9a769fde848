/*
 * moe_b200.h - C ABI of the B200 (sm_100a) routed mixture-of-experts layer with FP4 expert weights.
 *
 * The layer (paper, figure "Execution structure" and the accepted large-prefill path in the section
 * "Prefill optimization"): Router Top-k -> route production (expert sorter) -> FP4 routed experts
 * gate/up -> activation rounded to BF16 -> down projection, FP32 per-slot partials, unique-slot
 * stores -> fixed-order Top-k FP32 reduction.  One call per stage, in that order; moe_forward runs the
 * four stages as one call (one kernel launch for a single token), and moe_prepack re-lays the expert
 * weights once, byte for byte, for the *_packed forms of the calls that read them.
 *
 * Notation: T tokens, H hidden size, I expert intermediate size, E experts, k experts per token,
 * S = T*k slots, flat slot s = t*k + j (j = rank of the expert for token t, 0 = largest logit).
 *
 * Common rules
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer, 16-byte aligned, to a dense
 *     row-major array (innermost dimension contiguous).  The caller owns every buffer; the library
 *     allocates, frees and retains nothing.  `ws` is caller-provided scratch of at least
 *     moe_workspace_bytes() bytes, 256-byte aligned; its contents need not survive between calls
 *     and need no initialisation (moe_forward's workspace has one exception, stated there).
 *   - Every call only enqueues work on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *     legacy default stream) and returns; there is no host synchronisation and no device-to-host copy.
 *   - Return value: a moe_status_t.  Argument errors are found on the host before anything is
 *     launched.  A device-side bounded wait that runs out writes MOE_ERR_TIMEOUT to *status_word
 *     (sticky, device memory, may be NULL) and the kernel still terminates normally.  Once one wait of a
 *     call has run out (about two seconds), every later wait of that call gives up after a millisecond, so a
 *     lost signal costs seconds, not seconds per wait.  With status_word == NULL the kernels keep that rule
 *     through a word inside the library (one per device, looked up on the first such call on a device - make
 *     that call outside stream capture - and cleared by each call that uses it); nothing is reported then, and
 *     NULL-status calls that overlap on the GPU share the word.
 *   - Diagnostic and measurement exports (moe_debug_*) are declared in moe_b200_debug.h.
 *   - Determinism: identical inputs give bit-identical outputs on every launch.  No invariance is
 *     claimed across different T or batch compositions.
 *   - bf16 arrays are passed as `const void*` / `void*` (16-bit elements, IEEE bfloat16 bit patterns).
 *
 * FP4 weight format (the checkpoint's storage format, kept packed in HBM; paper, section on the
 * historical decode route: packed 4-bit weights without offline expansion, E2M1 nibbles, E8M0 scales)
 *   - codes: two E2M1 codes per byte along K, element 2j in bits 3:0 of byte j, element 2j+1 in bits 7:4.
 *     E2M1: bit 3 sign, bits 2:1 exponent (bias 1), bit 0 mantissa: magnitudes 0,.5,1,1.5,2,3,4,6.
 *   - scales: one E8M0 byte b per 32 consecutive K elements of a row, meaning 2^(b-127).
 *     The kernels support b in [0,128] (block scale up to 2); 255 (NaN) and 129..254 are rejected by
 *     moe_validate_scales and otherwise give unspecified values.
 *   - w13 [E, 2I, H/2] codes, rows [0,I) gate (w1), rows [I,2I) up (w3); w13_scale [E, 2I, H/32];
 *     w2 [E, H, I/2] codes; w2_scale [E, H, I/32].
 */
#ifndef MOE_B200_H_
#define MOE_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = 1,       /* null or misaligned pointer, non-positive size, k > E */
  MOE_ERR_UNSUPPORTED_SHAPE = 2, /* H or I not a multiple of 128, E > 1024, k > 32, T*k > 2^30 */
  MOE_ERR_WORKSPACE = 3,         /* ws is NULL, misaligned or too small; device side: moe_forward's counters not cleared */
  MOE_ERR_CUDA = 4,              /* a CUDA runtime call or a launch failed */
  MOE_ERR_TIMEOUT = 5            /* device side only: written to *status_word */
} moe_status_t;

typedef struct {
  int32_t T, H, I, E, k;
} moe_shape_t;

/* Host, pure.  Scratch bytes the four calls need for this shape (0 if the shape is unsupported). */
size_t moe_workspace_bytes(const moe_shape_t* shape);

/* Host, pure.  Static string for a moe_status_t value. */
const char* moe_status_string(int status);

/* Host.  Name of the kernel variant the calling thread's last successful moe_* call chose
 * (the choice is a pure function of the shape); "" before any call. */
const char* moe_last_kernel_name(void);

/* Host.  Number of kernels launched (memset nodes not counted) by this thread's moe_* calls so far. */
uint64_t moe_launch_count(void);

/*
 * Router Top-k (paper: "Router Top-k"; fixed Top-K membership and order is a stated requirement).
 *   logits [T,E] fp32 (finite).  For each token the k largest logits are selected, slot 0 the
 *   largest, equal logits in ascending expert id.  topk_w = softmax over the k selected logits,
 *   computed as e_j = EXP(l_j - l_0), s = ((e_0 + e_1) + ...) in fp32, w_j = e_j / s, where EXP is the
 *   fixed fp32 sequence: d = max(d,-80); n = rint(d*0x1.715476p+0f); r = fma(n,-0x1.62e4p-1f,d);
 *   r = fma(n,-0x1.7f7d1cp-20f,r); p = Horner/fma over 1/720,1/120,1/24,1/6,1/2,1,1 in r; EXP = p*2^n.
 *   expert_offsets [E+1] int32: exclusive prefix sum of the per-expert slot counts, [E] = T*k.
 * Launch order: for T <= 128 the kernel uses programmatic dependent launch.  It reads logits before it waits
 * for the kernel launched just before it on the stream, and writes its outputs only after that kernel has
 * completed (so the outputs of one layer call may be the buffers the previous call's moe_combine still reads).
 * If that preceding kernel releases its dependents early (cudaTriggerProgrammaticLaunchCompletion /
 * griddepcontrol.launch_dependents), logits must not be among its outputs; moe_combine's are not.
 * Errors: INVALID_ARG (null/misaligned, T<1, k<1, k>E), UNSUPPORTED_SHAPE (E>1024, k>32), WORKSPACE.
 */
int moe_route(const float* logits, int32_t T, int32_t E, int32_t k, int32_t* topk_ids /* [T,k] */,
              float* topk_w /* [T,k] */, int32_t* expert_offsets /* [E+1] */, void* ws, size_t ws_bytes,
              void* cuda_stream);

/*
 * Route production / expert sorter (paper: the sorter that groups assignments into per-expert row
 * blocks so an expert's packed weights are scanned once).  A stable counting sort of the flat slots
 * by expert id: perm[p] = slot at sorted position p (expert-major, ascending slot within an expert),
 * inv_perm[perm[p]] = p, x_perm[p,:] = x[perm[p]/k,:].
 *   x [T,H] bf16; topk_ids [T,k]; expert_offsets [E+1] as written by moe_route.
 */
int moe_permute(const void* x_bf16, const int32_t* topk_ids, const int32_t* expert_offsets,
                const moe_shape_t* shape, void* x_perm_bf16 /* [T*k,H] */, int32_t* perm /* [T*k] */,
                int32_t* inv_perm /* [T*k] */, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * FP4 routed experts: gate/up -> activation -> down (paper: stage 1, activation, stage 2).
 * For every expert e and sorted row p in [expert_offsets[e], expert_offsets[e+1]):
 *   g = W1_e x_p, u = W3_e x_p            (fp32 accumulation, weights = E2M1 value * 2^(scale-127))
 *   a = bf16_rne( silu(g) * u )           (the already-rounded BF16 intermediate; kept in ws)
 *   y_perm[p,:] = W2_e a                  (fp32, one store per (slot, column), no atomics)
 * The summation order inside a dot product is the kernel's; everything else is as written.
 *   status_word: device int32, may be NULL; see the common rules.
 * Three kernel variants, chosen by the shape alone (moe_last_kernel_name names the one that ran): for
 * decode-sized batches (T*k <= 32*E and <= 6144; H and I multiples of 256 up to 4096 - so also the I = 256 shard of
 * the paper's TP8 layout; E up to about 400 at H = 4096, where shared memory runs out) the packed weights feed the block-scaled FP4
 * tensor-core instruction directly and each bf16 activation row is written as a sum of eight E2M1 rows with their
 * own block scales (exact for elements within 2^-10 of their 32-block's largest magnitude; the others are off by
 * less than 2^-16 of that magnitude);
 * for prefill-sized batches (T*k >= 1024) weights are expanded to bf16 exactly on chip for a bf16 grouped GEMM;
 * every other supported shape uses a register-expansion streaming kernel.
 * Launch order: the decode-sized kernels use programmatic dependent launch.  They read expert_offsets and the
 * weights before waiting for the kernel launched just before them on the stream, and x_perm only after it has
 * completed: expert_offsets must not be written by that immediately preceding kernel (moe_permute does not).
 */
int moe_expert_ffn(const void* x_perm_bf16 /* [T*k,H] */, const int32_t* expert_offsets,
                   const uint8_t* w13, const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale,
                   const moe_shape_t* shape, float* y_perm /* [T*k,H] */, int32_t* status_word, void* ws,
                   size_t ws_bytes, void* cuda_stream);

/*
 * Fixed-order Top-k FP32 reduction (paper: the vectorised fixed-order Top-k FP32 reducer that
 * replaces cross-expert atomics).  out[t,n] = bf16_rne(acc_k), acc_0 = 0,
 * acc_{j+1} = fma(topk_w[t,j], y_perm[inv_perm[t*k+j], n], acc_j), j = 0..k-1 ascending.
 */
int moe_combine(const float* y_perm, const int32_t* inv_perm, const float* topk_w, const moe_shape_t* shape,
                void* out_bf16 /* [T,H] */, void* cuda_stream);

/*
 * One-time load check of E8M0 scale bytes (paper: scale layout and value traps, "test real
 * nonconstant scales").  Counts bytes outside [0,128] into *bad_count (device int32, overwritten).
 */
int moe_validate_scales(const uint8_t* scales, size_t n_bytes, int32_t* bad_count, void* cuda_stream);

/*
 * One-time load transform of the expert weights, and moe_expert_ffn on its result.  The paper applies transforms of
 * this kind when a checkpoint is loaded (its section on load-time weight layouts) and warns that the scales must
 * follow the same address map as the codes and that expanded weights cost more traffic than they save: here the
 * packed buffer holds exactly the same bytes (4.25 bits per weight; moe_prepack_bytes() = the four tensors' sizes
 * rounded up to 256 bytes each), in another order.
 *
 *   - Layout (private to the library; for H and I multiples of 512): the codes of 128 consecutive rows x 128
 *     consecutive bytes (256 K elements) form one contiguous 16 KB tile, the tiles of a row block following each other
 *     along K; the scale bytes likewise in tiles of 128 rows x 16 bytes.  A kernel's pipeline step then reads whole
 *     contiguous runs instead of 128 pieces one row pitch apart.  For every other shape the packed buffer is a plain
 *     copy of the four tensors.
 *   - moe_prepack: device to device, out of place (packed_out must not overlap the inputs), 256-byte aligned,
 *     packed_bytes >= moe_prepack_bytes() else MOE_ERR_WORKSPACE.  Not part of the timed path: weights are packed once
 *     per model load.  It is also the load check of the scale bytes (the paper's scale-value trap): both scale
 *     tensors are scanned for bytes outside [0,128], the count is read back, and MOE_ERR_INVALID_ARG is returned -
 *     with nothing packed - if there is one.  Because of that read-back this call, unlike the others, WAITS for the
 *     stream and cannot be captured into a CUDA graph.  The caller may free the four tensors afterwards.
 *   - moe_expert_ffn_packed: moe_expert_ffn with `packed` in place of the four weight arguments; same arithmetic, same
 *     result bit for bit.  Kernel choice as moe_expert_ffn, except that shapes with the tiled layout that would fall to
 *     the row-streaming fallback kernel (neither decode-sized nor prefill-sized) run the grouped-GEMM kernel.
 */
size_t moe_prepack_bytes(const moe_shape_t* shape);
int moe_prepack(const uint8_t* w13, const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale,
                const moe_shape_t* shape, void* packed_out, size_t packed_bytes, void* cuda_stream);
int moe_expert_ffn_packed(const void* x_perm_bf16 /* [T*k,H] */, const int32_t* expert_offsets, const void* packed,
                          const moe_shape_t* shape, float* y_perm /* [T*k,H] */, int32_t* status_word, void* ws,
                          size_t ws_bytes, void* cuda_stream);

/*
 * The whole layer in one call on DEVICE buffers: route -> permute -> expert_ffn -> combine of the same inputs, with
 * every intermediate (sorted rows, per-slot outputs) kept in `ws`.  The paper's own decode gains came from cutting
 * passes and launches around the expert kernels (its optimisation history and the section on the down-projection
 * consumer); this is that step for this library.  Result: out [T,H] bf16 exactly as moe_combine would write it after
 * the three calls before it, and - where the pointers are not NULL - topk_ids / topk_w [T,k] exactly as moe_route
 * writes them.
 *
 *   - For T = 1 (k <= 32, E*4 <= 4*max(H,I) bytes) on shapes the decode-sized expert kernel takes,
 *     the call is ONE kernel launch: every CTA routes the token itself and sorts the slots, the first CTAs write the
 *     token's E2M1 term rows, every CTA runs its share of the gate/up and down items, and the CTA that finishes a
 *     column tile's last expert reduces that tile over the slots.  Any other shape runs the four calls back to back
 *     (from two tokens on they are the faster form).
 *   - ws: moe_forward_workspace_bytes() bytes, 256-byte aligned.  Its first moe_forward_sync_bytes() bytes are the
 *     kernel's completion counters: they must be ZERO when a call starts.  Clear them once (cudaMemsetAsync) before
 *     the first call that uses this ws; every call that returns MOE_OK and whose kernels ran to completion leaves them
 *     zero, also when *status_word reports a device-side timeout.  The rest of ws is scratch.  Calls that share a ws
 *     must be ordered on one stream.  Two words of the block are never written by any kernel; a one-launch call that
 *     finds one of them non-zero writes MOE_ERR_WORKSPACE to *status_word and leaves `out` untouched (this catches a block
 *     that was never cleared, not one that was cleared and then damaged).
 *   - Asynchronous, no allocation, capturable into a CUDA graph, bounded device-side waits as moe_expert_ffn.
 */
size_t moe_forward_workspace_bytes(const moe_shape_t* shape);
size_t moe_forward_sync_bytes(void);
int moe_forward(const float* logits /* [T,E] */, const void* x_bf16 /* [T,H] */, const uint8_t* w13, const uint8_t* w13_scale,
                const uint8_t* w2, const uint8_t* w2_scale, const moe_shape_t* shape, void* out_bf16 /* [T,H] */,
                int32_t* topk_ids /* [T,k] or NULL */, float* topk_w /* [T,k] or NULL */, int32_t* status_word, void* ws,
                size_t ws_bytes, void* cuda_stream);
/* The same on weights written by moe_prepack (same workspace, same rules, same result). */
int moe_forward_packed(const float* logits /* [T,E] */, const void* x_bf16 /* [T,H] */, const void* packed,
                       const moe_shape_t* shape, void* out_bf16 /* [T,H] */, int32_t* topk_ids /* [T,k] or NULL */,
                       float* topk_w /* [T,k] or NULL */, int32_t* status_word, void* ws, size_t ws_bytes,
                       void* cuda_stream);

/*
 * moe_forward with HOST input and output for one batch: copies logits_host [T,E] and x_host [T,H] to
 * device buffers carved from `ws`, clears moe_forward's counters, runs moe_forward on `cuda_stream`,
 * copies out [T,H] bf16 back into out_host and waits for the stream.  Fewer stream operations where the sizes allow: an
 * output of at most 64 KB in page-locked memory that the device can address is written there by the last kernel itself;
 * a single token row in such memory is read there by the kernel; logits of at most 64 KB travel in one copy with the
 * zeros of moe_forward's counter block, through a page-locked staging buffer that the library allocates once per host
 * thread (the only allocation any entry point makes, on its first call).
 * Weights stay device-resident (they are model state, not per-batch input).  For page-locked host
 * buffers the copies are asynchronous until the final wait.  ws must hold
 * moe_forward_host_workspace_bytes() bytes.  No counterpart in the paper: it is the end-to-end
 * measurement path of the layer.
 */
size_t moe_forward_host_workspace_bytes(const moe_shape_t* shape);
int moe_forward_host(const float* logits_host, const void* x_host_bf16, const uint8_t* w13,
                     const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale,
                     const moe_shape_t* shape, void* out_host_bf16, int32_t* status_word, void* ws,
                     size_t ws_bytes, void* cuda_stream);
/* The same on weights written by moe_prepack. */
int moe_forward_host_packed(const float* logits_host, const void* x_host_bf16, const void* packed,
                            const moe_shape_t* shape, void* out_host_bf16, int32_t* status_word, void* ws,
                            size_t ws_bytes, void* cuda_stream);

/*
 * The steps either side of the routed path (paper, figure "Execution structure": router scores before the Top-k; the
 * shared expert beside the routed experts; "add partials" after them), and the FFN block they make with it.
 *
 *   - moe_router_logits: logits[t,e] = sum_h x[t,h] * w_router[e,h]; x [T,H] and w_router [E,H] bf16, fp32
 *     accumulation (each product is exact in fp32; the order of the sum is the kernel's), logits [T,E] fp32.  The paper
 *     states no precision for this step (it kept a vendor BLAS).  H a multiple of 128, E <= 1024.  Up to 16 tokens: one
 *     warp per expert streams w_router once; more: a tcgen05 GEMM on tiles of 128 tokens x 64 experts.
 *   - The shared expert is one more expert in the routed experts' weight format, applied to every token with weight 1:
 *     tensors shaped as the routed ones with E = 1.  It needs no entry point of its own: moe_expert_ffn with x as
 *     x_perm, offsets {0, T} and shape {T, H, I, 1, 1} gives y_shared [T,H] fp32.
 *   - moe_combine_shared: out[t,n] = bf16_rne( acc_k + y_shared[t,n] ), acc as in moe_combine (fma over the slots in slot
 *     order from zero), then one fp32 addition, then one rounding.
 *   - moe_ffn_block: router projection -> moe_route -> moe_permute -> moe_expert_ffn (routed) -> moe_expert_ffn (shared)
 *     -> moe_combine_shared on DEVICE buffers, every intermediate in `ws` (moe_ffn_block_workspace_bytes(), 256-byte
 *     aligned, no initialisation needed).  topk_ids / topk_w [T,k] receive the routing where not NULL.  Enqueue only,
 *     no allocation, capturable, bounded device-side waits.  One token (on shapes moe_forward runs as one launch, with
 *     room for one more expert's CTAs): the router projection, then one launch - the shared expert is an extra slot of
 *     the one-token kernel, added with weight 1 after the routed slots (the same order of operations).
 */
int moe_router_logits(const void* x_bf16 /* [T,H] */, const void* w_router_bf16 /* [E,H] */, int32_t T, int32_t H, int32_t E,
                      float* logits /* [T,E] */, int32_t* status_word, void* cuda_stream);
int moe_combine_shared(const float* y_perm, const int32_t* inv_perm, const float* topk_w, const float* y_shared /* [T,H] */,
                       const moe_shape_t* shape, void* out_bf16 /* [T,H] */, void* cuda_stream);
size_t moe_ffn_block_workspace_bytes(const moe_shape_t* shape);
int moe_ffn_block(const void* x_bf16 /* [T,H] */, const void* w_router_bf16 /* [E,H] */, const uint8_t* w13,
                  const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale, const uint8_t* shared_w13 /* [1,2I,H/2] */,
                  const uint8_t* shared_w13_scale, const uint8_t* shared_w2 /* [1,H,I/2] */, const uint8_t* shared_w2_scale,
                  const moe_shape_t* shape, void* out_bf16 /* [T,H] */, int32_t* topk_ids /* [T,k] or NULL */,
                  float* topk_w /* [T,k] or NULL */, int32_t* status_word, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Quantised-activation variant of moe_expert_ffn (paper, "historical TP4/EP1 decode route": the BF16 activations are
 * quantised online, one scale per 32 elements, so that a low-precision dot product consumes them; the paper's target is
 * INT8, this library's is the weights' own format, which the block-scaled FP4 tensor-core instruction takes directly).
 *
 *   - Quantiser, applied to every row of x_perm along H and to every row of the bf16 intermediate along I, per block of
 *     32 consecutive elements: amax = max |v|; s = the smallest integer in [-126, 126] with amax <= 6 * 2^s (s = 0 for
 *     an all-zero block); code = E2M1 value nearest to v / 2^s, ties to the even code; the contraction consumes
 *     E2M1(code) * 2^s.  Everything else as moe_expert_ffn: g, u in fp32, act = bf16_rne(silu(g) * u), y_perm fp32.
 *     Inputs with |v| > 2^126 are outside the domain.
 *   - Result: y_perm differs from moe_expert_ffn's by the quantisation error (about a quarter of the output's norm on
 *     the benchmark's inputs: one E2M1 term keeps two to three significant bits); against this variant's own oracle the
 *     result is the same - bit for bit on most rows - up to fp32 summation order, the fast exponential and division of the
 *     SwiGLU, and the roundings those can flip: about one row in two hundred has one element of its intermediate one code
 *     step away from the oracle's.
 *   - Weights: the four logical tensors with packed = NULL, or packed = the buffer of moe_prepack with the four NULL.
 *   - Shapes: H and I multiples of 256 and at most 4096; otherwise MOE_ERR_UNSUPPORTED_SHAPE.  Any T * k: one kernel
 *     serves decode and prefill (a pass holds 128 tokens of an expert, against 16 in moe_expert_ffn's kernel).
 *   - `ws`: moe_expert_ffn_q_workspace_bytes(), 256-byte aligned, no initialisation needed.  Enqueue only, no
 *     allocation, capturable, bounded device-side waits and status_word as moe_expert_ffn.
 */
size_t moe_expert_ffn_q_workspace_bytes(const moe_shape_t* shape);
int moe_expert_ffn_q(const void* x_perm_bf16 /* [T*k,H] */, const int32_t* expert_offsets, const uint8_t* w13,
                     const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale, const void* packed,
                     const moe_shape_t* shape, float* y_perm /* [T*k,H] */, int32_t* status_word, void* ws, size_t ws_bytes,
                     void* cuda_stream);

/*
 * Expert-parallel sharding of the routed layer over `world` GPUs, one process each (the paper compares a tensor-parallel
 * layout with expert-parallel ones, "TP8/EP1" against "TP4/EP4"; outside the single-GPU workloads this library is
 * measured on).  Rank r holds the weights of the experts [e_begin, e_end) and finishes the tokens
 * [r * tpr, (r + 1) * tpr), tpr = ceil(T / world).  Every rank runs moe_route and moe_ep_permute on ALL tokens (identical
 * routing and order everywhere); its experts' rows are one contiguous range of the sorted order.  Then
 *   - moe_ep_row_table fills row_dst[p], for the sorted rows p of this rank's experts, with the address of row
 *     (token - owner * tpr) * k + slot of owner_y[owner], owner = token / tpr: owner_y is a DEVICE array of `world`
 *     pointers to the ranks' buffers [tpr * k, H] fp32 - peer memory for the other ranks (the caller maps it: CUDA IPC,
 *     symmetric memory; the library only stores through the pointers);
 *   - moe_ep_expert_ffn is moe_expert_ffn on this rank's experts (weights [e_end - e_begin, ...], the GLOBAL
 *     expert_offsets and shape), whose down projection stores every output row through row_dst instead of into a local
 *     y_perm: the exchange ("combine" in expert-parallel terms) happens in the kernel's epilogue, row by row;
 *   - after a barrier between the ranks (the caller's: all stores of all ranks complete), each rank runs moe_combine on
 *     its buffer with the identity as inv_perm and its tokens' rows of topk_w: the same fp32 rows in the same slot order
 *     as on one GPU, so the result is bit-identical to the unsharded layer.
 * e_begin must be a multiple of 4 (alignment of the shifted offsets); `ws` as for moe_expert_ffn on the global shape.
 * Enqueue only, no allocation, capturable, bounded device-side waits; no kernel of one rank waits for another rank.
 */
/* moe_permute of which a rank needs the order (perm, inv_perm: complete) but only its own experts' rows of x_perm: for
 * batches of more than 4096 slots only those rows are copied (smaller batches: all, the copy is part of one small kernel) */
int moe_ep_permute(const void* x_bf16, const int32_t* topk_ids, const int32_t* expert_offsets, const moe_shape_t* shape,
                   int32_t e_begin, int32_t e_end, void* x_perm_bf16, int32_t* perm, int32_t* inv_perm, void* ws,
                   size_t ws_bytes, void* cuda_stream);
int moe_ep_row_table(const int32_t* perm, const int32_t* expert_offsets, const moe_shape_t* shape, int32_t e_begin,
                     int32_t e_end, float* const* owner_y /* device, [world] */, int32_t world,
                     float** row_dst /* device, [T*k] */, void* cuda_stream);
int moe_ep_expert_ffn(const void* x_perm_bf16 /* [T*k,H] */, const int32_t* expert_offsets /* [E+1], all experts */,
                      const uint8_t* w13_local, const uint8_t* w13_scale_local, const uint8_t* w2_local,
                      const uint8_t* w2_scale_local, const moe_shape_t* shape /* global */, int32_t e_begin, int32_t e_end,
                      float* const* row_dst /* device, [T*k] */, int32_t* status_word, void* ws, size_t ws_bytes,
                      void* cuda_stream);

/*
 * moe_expert_ffn without a workspace argument, for callers that cannot allocate device memory
 * (the paper has no counterpart: this is a packaging variant of moe_expert_ffn, same arithmetic).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plug-in called inside another
 * framework's stream-ordered or graph-managed section, a real-time loop that must not touch the driver's
 * allocator, a host that hands this library pre-made buffers for inputs and outputs only.  Such a caller
 * still passes every input and output, but not the scratch: what the kernels keep between their launches sits
 * in a fixed array of moe_expert_ffn_noalloc_max_bytes() = 16 MiB inside the library image (each GPU that loads
 * the library holds those 16 MiB until the process exits).
 *
 *   - Sizes: the bf16 intermediate (2*T*k*I bytes) - for the decode-sized kernel variant the E2M1 term rows of
 *     both projections' inputs, 4.25*T*k*(H+I) bytes - must fit the array, else MOE_ERR_WORKSPACE and nothing is
 *     launched (up to 640 slots at H = 4096, I = 2048).  Other argument rules as moe_expert_ffn.
 *   - The call allocates and frees nothing and calls no allocating library routine.  Its first call on a
 *     device looks up the array's device address (one runtime query, cached per device): make that first
 *     call outside any stream capture.
 *   - All calls share the one array and it keeps the last call's contents.  Nothing in it needs to start
 *     at zero (each call writes every row it later reads), but two calls that overlap on the GPU - other
 *     streams, other host threads - race on it: keep calls on one stream or order them yourself.
 *   - Result: identical to moe_expert_ffn on the same inputs (same kernels, same kernel choice).
 */
size_t moe_expert_ffn_noalloc_max_bytes(void);
int moe_expert_ffn_noalloc(const void* x_perm_bf16 /* [T*k,H] */, const int32_t* expert_offsets, const uint8_t* w13,
                           const uint8_t* w13_scale, const uint8_t* w2, const uint8_t* w2_scale,
                           const moe_shape_t* shape, float* y_perm /* [T*k,H] */, int32_t* status_word,
                           void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H_ */
