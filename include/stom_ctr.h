/*
 * stom_ctr.h -- C ABI of the Causal Temporal Reduction (CTR) steps that
 * libstom_oqm.so implements: the part of StreamingTOM that runs BEFORE the
 * language model and decides which G of a frame's N vision tokens are kept
 * (paper Sec. 3.3).  Built here: the per-token temporal similarity, the
 * static / dynamic split, the proportional budget and the saliency selection
 * of the dynamic tokens.  NOT built: Merge_{k_s}, the density-based clustering
 * of the static tokens -- the paper names it but gives no definition of it.
 *
 * Conventions are those of stom_oqm.h: device pointers unless stated, caller
 * owns all memory, work is enqueued on `stream` without synchronising, return
 * value STOM_OK or a negative STOM_ERR_* code, argument errors are found on
 * the host before anything is launched, inputs must be finite.
 */
#ifndef STOM_CTR_H
#define STOM_CTR_H

#include <stdint.h>

#include "stom_oqm.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Sec. 3.3, the s_t^(i) equation: cosine similarity of every token of frame t
 * with the token at the same position of frame t-1, for the T frames of one
 * call.
 *   F      element (t, i, c) at t*stride_frame + i*stride_token + c (strides in
 *          elements; the channel axis is contiguous), T frames x N tokens x D
 *          channels of type `dtype` (STOM_BF16 | STOM_FP16 | STOM_FP32)
 *   prev   nullable: the frame before F[0], [N][D] with the same token stride
 *          -- the only state the method carries between calls.  NULL: frame 0
 *          is the first of its stream, has no predecessor, and gets -inf
 *          (none of its tokens is static)
 *   sim    out, [T][N] float.  A zero vector has similarity 0 (each norm is
 *          clamped below by 1e-12).  Accumulation is binary32.
 * D must be a multiple of 8 (of 4 for STOM_FP32), at most 4096 (2048 for
 * STOM_FP32: a row of at most 8 KB); rows must start 16-byte aligned.
 * Errors: INVALID_ARG, SHAPE (D, N out of range), ALIGNMENT, UNSUPPORTED
 * (dtype), CUDA.
 */
int32_t stom_ctr_similarity(const void *F, const void *prev, int32_t dtype, int32_t T, int32_t N, int32_t D,
                            int64_t stride_frame, int64_t stride_token, float *sim, void *stream);

/*
 * Sec. 3.3, the (S_t, D_t) equation, the (k_s, k_d) equation and the TopK
 * half of the (G_d, G_s) equation, per frame:
 *   S_t = {i : sim[t][i] > tau_c},  D_t = the other tokens
 *   k_s = floor(G |S_t| / N),  k_d = G - k_s
 *   G_d = the k_d tokens of D_t with the largest saliency alpha[t][i]; equal
 *         saliencies resolve to the lower token index
 *   sim, alpha  [T][N] float (alpha: the vision encoder's attention-based
 *               saliency in [0, 1], an input)
 *   k_s, k_d    out, [T] int32
 *   static_idx  out, [T][N] int32: S_t in ascending order, unused slots -1
 *               (what Merge_{k_s} would consume)
 *   dyn_idx     out, [T][G] int32: G_d in ascending order, unused slots -1
 * 1 <= G <= N <= 1024.  Errors: INVALID_ARG, SHAPE, ALIGNMENT, CUDA.
 */
int32_t stom_ctr_select(const float *sim, const float *alpha, int32_t T, int32_t N, int32_t G, float tau_c,
                        int32_t *k_s, int32_t *k_d, int32_t *static_idx, int32_t *dyn_idx, void *stream);

/*
 * Both steps for the T frames of one call, back to back on `stream`:
 * stom_ctr_similarity into `sim`, then stom_ctr_select from it.  Arguments
 * and errors as above.
 */
int32_t stom_ctr_reduce(const void *F, const void *prev, int32_t dtype, int32_t T, int32_t N, int32_t D,
                        int64_t stride_frame, int64_t stride_token, const float *alpha, int32_t G, float tau_c,
                        float *sim, int32_t *k_s, int32_t *k_d, int32_t *static_idx, int32_t *dyn_idx, void *stream);

#ifdef __cplusplus
}
#endif

#endif /* STOM_CTR_H */
