/*
 * tsp_attn.h - C ABI of the projection GEMMs of TSP attention (same library as tsp_mlp.h, B200 / sm_100a).
 *
 * Algorithm 1 (TSP multi-head attention, forward pass on rank p) loops over the D weight-owning ranks r; in
 * every iteration a rank projects its own tokens with shard r of the weights,
 *     Q = X W_Q^(r)T,  K = X W_K^(r)T,  V = X W_V^(r)T        W_Q^(r) in R^{(h/D) x h}; GQA: K/V shards h/(gD) wide
 * and, after attention on those heads, adds their output through shard r of the output projection,
 *     Y <- Y + Flatten(A) W_O^(r)T                             W_O^(r) in R^{h x (h/D)},  Y starts at 0.
 * These entry points compute the two dense steps for all D shards resident on ONE GPU (no broadcast, no
 * collective), forward and backward; the attention core between them is not part of this library.
 *
 * Layouts (DEVICE pointers, row-major bf16, inputs 16-byte aligned, outputs 32-byte aligned):
 *     X        [S, H]               tokens of every rank (the projections are row-wise: any token order)
 *     Wq       [D][Hq/D][H]         shard r = rows of heads r*H_s .. (r+1)*H_s-1  (= the ordinary [Hq, H] matrix)
 *     Wk, Wv   [D][Hkv/D][H]        Hkv = Hq / g
 *     Q        [S, Hq]              heads side by side: shard r's heads are columns r*Hq/D .. (r+1)*Hq/D
 *     K, V     [S, Hkv]
 *     A        [S, Hq]              attention output, same column layout as Q
 *     Wo       [D][H][Hq/D]         shard r = W_O^(r), the columns of Wo that multiply shard r's heads
 *     Y        [S, H]
 * Shapes: H % 256 == 0, Hq % 256 == 0, Hkv % 256 == 0, Hq % D == 0, Hkv % D == 0, (Hq/D) % 64 == 0, 1 <= D <= 64,
 * 1 <= S <= 2^24 (any S: the last token tile is loaded whole and only its valid rows are stored).
 * Arithmetic: bf16 inputs, fp32 accumulation in tensor memory, one round-to-nearest-even to bf16 per output.
 * Status codes, asynchrony, ownership and threading rules are those of tsp_mlp.h; nothing is allocated per call
 * and no workspace is needed.
 */
#ifndef TSP_ATTN_H
#define TSP_ATTN_H

#include "tsp_mlp.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tsp_attn_plan tsp_attn_plan_t; /* opaque; created by tsp_attn_plan, owned by the library */

/*
 * tsp_attn_plan - validate (H, Hq, Hkv, D) for the current device (inputs of Algorithm 1: hidden size, head
 * widths, world size) and build a plan; release it with tsp_attn_plan_destroy.  Allocates a small device control
 * block (status word, tile-scheduler words).  Errors: INVALID_ARG, UNSUPPORTED_SHAPE, UNSUPPORTED_DEVICE, CUDA.
 */
tsp_status_t tsp_attn_plan(int H, int Hq, int Hkv, int D, tsp_attn_plan_t** out);
tsp_status_t tsp_attn_plan_destroy(tsp_attn_plan_t* plan);

/*
 * tsp_attn_qkv_forward - the "local projections" line of Algorithm 1 for all D shards: Q = X Wq^T, K = X Wk^T,
 * V = X Wv^T.  One kernel (tcgen05 CTA-pair GEMM over the concatenated output features).  `D` must equal the
 * plan's.  Errors: INVALID_ARG (null / misaligned pointer, D mismatch, S < 1), UNSUPPORTED_SHAPE (S > 2^24), CUDA.
 */
tsp_status_t tsp_attn_qkv_forward(tsp_attn_plan_t* plan, const void* X, const void* Wq, const void* Wk, const void* Wv,
                                  void* Q, void* K, void* V, int64_t S, int D, void* cuda_stream);

/*
 * tsp_attn_out_forward - the "output projection + accumulate" line of Algorithm 1 over all D iterations:
 * Y = sum_{r=0..D-1} A[:, shard r] Wo^(r)T, accumulated in fp32 tensor memory in the order of the loop (r ascending,
 * the same on every rank), one bf16 store of Y (no all-reduce over activations: every rank applies every shard to
 * its own tokens).  One kernel.  Errors as above.
 */
tsp_status_t tsp_attn_out_forward(tsp_attn_plan_t* plan, const void* A, const void* Wo, void* Y, int64_t S, int D,
                                  void* cuda_stream);

/*
 * Backward of the two steps (the backward pass mirrors the forward weight movement; the partial weight gradients
 * the ranks produce for a shard are summed to its owner: Sections 4.3.4 and 4.7 - here all ranks' tokens are
 * resident, so the sum over ranks is the contraction over all S tokens, in ascending token order).
 *
 * tsp_attn_qkv_backward: for upstream dQ [S, Hq], dK, dV [S, Hkv] (bf16):
 *     dX  = dQ Wq + dK Wk + dV Wv                [S, H] bf16 (fp32 accumulation over all features, one rounding)
 *     dWq = dQ^T X, dWk = dK^T X, dWv = dV^T X   fp32, in the layouts of Wq, Wk, Wv, overwritten
 *   Two kernels.
 * tsp_attn_out_backward: for upstream dY [S, H] (bf16):
 *     dA  = dY Wo                                [S, Hq] bf16, heads of shard r in columns r*Hq/D ..
 *     dWo = dY^T A                               fp32 [D][H][Hq/D], overwritten
 *   Two kernels.
 * Errors as for the forward calls; fp32 outputs must be 32-byte aligned.
 */
tsp_status_t tsp_attn_qkv_backward(tsp_attn_plan_t* plan, const void* X, const void* Wq, const void* Wk, const void* Wv,
                                   const void* dQ, const void* dK, const void* dV, void* dX, float* dWq, float* dWk,
                                   float* dWv, int64_t S, int D, void* cuda_stream);
tsp_status_t tsp_attn_out_backward(tsp_attn_plan_t* plan, const void* A, const void* Wo, const void* dY, void* dA,
                                   float* dWo, int64_t S, int D, void* cuda_stream);

/* Device status word (after the stream has been synchronized): TSP_OK or TSP_ERR_DEVICE_TIMEOUT; clears it. */
tsp_status_t tsp_attn_status(tsp_attn_plan_t* plan);

/* Per-kernel timing with CUDA events on the launch stream, as tsp_mlp_profile_*: a forward call records one
 * kernel, a backward call two; ms_out must have room for 8 floats. */
tsp_status_t tsp_attn_profile_begin(tsp_attn_plan_t* plan, int max_calls);
tsp_status_t tsp_attn_profile_read(tsp_attn_plan_t* plan, int call_index, int* n_kernels_out, float* ms_out);
tsp_status_t tsp_attn_profile_end(tsp_attn_plan_t* plan);

#ifdef __cplusplus
}
#endif
#endif /* TSP_ATTN_H */
