/*
 * stom_ctr.h -- C ABI of the Causal Temporal Reduction (CTR) steps that
 * libstom_oqm.so implements: the part of StreamingTOM that runs BEFORE the
 * language model and decides which G of a frame's N vision tokens are kept
 * (paper Sec. 3.3): the per-token temporal similarity, the static / dynamic
 * split, the proportional budget, the saliency selection of the dynamic
 * tokens, the consolidation of the static tokens (Merge_{k_s}) and the
 * retained group of G tokens that goes on to the language model.  The paper
 * specifies all of these but the clustering inside Merge_{k_s}, which it only
 * names (a density-based clustering); the rule used here is written out at
 * stom_ctr_merge and is this library's reading, not the paper's text.
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
 *               (what stom_ctr_merge consumes)
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

/*
 * Sec. 3.3, the Merge half of the (G_d, G_s) equation, G_s = Merge_{k_s}({F_t^(i)}, i in S_t), and the retained
 * group G_t of Sec. 3.3 (the selected dynamic tokens and the merged static ones together, |G_t| = G), per frame.
 *
 * The paper consolidates the static tokens by a density-based clustering (density peaks, going by its overview
 * figure) and gives neither the density, nor the distance, nor how a cluster becomes one token.  This library's
 * reading -- the k-nearest-neighbour form of density-peak clustering -- over the n_s static tokens x_i of a frame:
 *   d2(i,j) = |x_i - x_j|^2 / D                                   (computed as (|x_i|^2 + |x_j|^2 - 2 x_i.x_j) / D
 *                                                                  in binary32, clamped at 0)
 *   rho_i   = exp(-(1/kk) * sum of the kk smallest d2(i,j), j != i),  kk = min(knn, n_s - 1)  (kk = 0: rho = 1)
 *   delta_i = min d(i,j) over the denser tokens j (rho_j > rho_i, or equal and j earlier), d = sqrt(d2);
 *             the densest token of all takes its largest distance
 *   the k_s tokens of largest rho_i * delta_i are the centres (equal products: the earlier token)
 *   every other static token joins its nearest centre (equal distances: the earlier centre)
 *   a cluster becomes ONE token: the mean of its members' features (binary32 sums in ascending token order, the
 *   correctly rounded binary32 quotient), rounded to the feature type, standing at its centre's position
 * Retained group: the k_d selected dynamic rows, copied unchanged, and the k_s merged rows, in ascending position.
 *   F            as for stom_ctr_similarity; dtype STOM_BF16 or STOM_FP16 (the Gram matrix runs on the tensor cores)
 *   k_s, k_d, static_idx, dyn_idx   the outputs of stom_ctr_select for the same T frames
 *   knn          neighbours in the density, 0 .. 8 (5 is the usual choice)
 *   retained     out, [T][G][D] of dtype; rows behind the k_d + k_s tokens of a frame are zero
 *   retained_pos out, [T][G] int32: token position of every retained row, -1 behind them
 *   centre       out, nullable, [T][G] int32: the centres in ascending order, -1 padded
 *   assign       out, nullable, [T][N] int32: for the a-th static token the index of its cluster in `centre`, -1 padded
 *   dev_flags    nullable device word: STOM_FLAG_TIMEOUT is OR-ed in when a tensor-core product of a frame had not
 *                completed after 0.1 s (that frame's outputs are then undefined; nothing traps, the call ends)
 * 1 <= G <= N <= 224, D a multiple of 64, at most 8192.  Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALIGNMENT, CUDA.
 */
int32_t stom_ctr_merge(const void *F, int32_t dtype, int32_t T, int32_t N, int32_t D, int64_t stride_frame,
                       int64_t stride_token, const int32_t *k_s, const int32_t *k_d, const int32_t *static_idx,
                       const int32_t *dyn_idx, int32_t G, int32_t knn, void *retained, int32_t *retained_pos,
                       int32_t *centre, int32_t *assign, uint32_t *dev_flags, void *stream);

/*
 * The whole of CTR for the T frames of one call, back to back on `stream`: stom_ctr_reduce (similarity, split,
 * budget, saliency selection), then stom_ctr_merge.  What comes out in `retained` is the [T][G][D] token stream the
 * language model consumes; with the model's K and V of those tokens, stom_oqm_quantize_frame takes over.
 * Arguments and errors as above.
 */
int32_t stom_ctr_reduce_tokens(const void *F, const void *prev, int32_t dtype, int32_t T, int32_t N, int32_t D,
                               int64_t stride_frame, int64_t stride_token, const float *alpha, int32_t G, float tau_c,
                               int32_t knn, float *sim, int32_t *k_s, int32_t *k_d, int32_t *static_idx,
                               int32_t *dyn_idx, void *retained, int32_t *retained_pos, uint32_t *dev_flags,
                               void *stream);

#ifdef __cplusplus
}
#endif

#endif /* STOM_CTR_H */
