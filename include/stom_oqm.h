/*
 * stom_oqm.h -- C ABI of libstom_oqm.so: StreamingTOM's Online Quantized
 * Memory (OQM) on NVIDIA B200 (sm_100a).
 *
 * The library implements the post-LLM path of the method: 4-bit group
 * quantization of each arriving frame's retained-token kv-cache, cosine
 * scoring of the stored groups against the question embedding, top-K group
 * selection, and dequantize-and-gather of the selected groups into the
 * bounded active kv-cache (plus a decode attention that dequantizes on the
 * fly).  A "group" is the G tokens one frame keeps; it is the atomic unit of
 * storage and of retrieval (paper Sec. 3.2 and Sec. 3.4).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers unless a parameter is documented
 *     as "host".  Structs (config, store descriptor) are read on the host.
 *   - The caller owns all memory.  The library allocates nothing on the
 *     device, keeps no state between calls and never frees anything; two
 *     calls may run concurrently on different streams if their outputs do
 *     not overlap.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and the call returns without synchronising.
 *   - Return value: STOM_OK or a negative STOM_ERR_* code.  Argument errors
 *     are found on the host before anything is launched.  Device-resident
 *     indices that are out of range are skipped by the kernels, which set a
 *     bit in the optional `dev_flags` word instead of trapping.
 *   - Inputs must be finite.  Strides are in ELEMENTS of the tensor's type;
 *     the channel axis is always contiguous (stride 1).
 *   - Alignment: every base pointer 16-byte aligned; every stride such that
 *     a row of head_dim elements starts 16-byte aligned.
 */
#ifndef STOM_OQM_H
#define STOM_OQM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ---------------------------------------------------- */
#define STOM_OK 0
#define STOM_ERR_INVALID_ARG (-1) /* null pointer, negative count, bad range          */
#define STOM_ERR_SHAPE (-2)       /* geometry the kernels do not cover                */
#define STOM_ERR_ALIGNMENT (-3)   /* pointer or stride breaks the 16-byte rule        */
#define STOM_ERR_CAPACITY (-4)    /* group range beyond capacity_groups               */
#define STOM_ERR_INDEX (-5)       /* host-visible index out of range                  */
#define STOM_ERR_UNSUPPORTED (-6) /* bits / dtype / mode not implemented              */
#define STOM_ERR_CUDA (-7)        /* launch failed; see stom_last_cuda_error()        */
#define STOM_ERR_WORKSPACE (-8)   /* workspace missing or too small                   */
#define STOM_ERR_NOALLOC_LIMIT (-9) /* request exceeds the built-in scratch of a *_noalloc call */

/* ---- element types and modes ----------------------------------------- */
#define STOM_BF16 0
#define STOM_FP16 1
#define STOM_FP32 2

/* appendix "Question-guided single-pass retrieval": one selection per layer
 * over the kv heads flattened into one vector (PER_LAYER, the paper's rule);
 * PER_HEAD keeps the heads apart (one selection per layer and kv head). */
#define STOM_SCORE_PER_LAYER 0
#define STOM_SCORE_PER_HEAD 1

/* bits of dev_flags set by kernels */
#define STOM_FLAG_BAD_INDEX 1u /* an entry of idx was < -1 or >= n_groups and was skipped */
#define STOM_FLAG_TIMEOUT 2u   /* a bounded wait inside a kernel ran out; the call's outputs are incomplete */
#define STOM_FLAG_DIRTY_WORKSPACE 4u /* reserved: raised by an earlier form of stom_oqm_attend that kept counters in a
                                        caller-cleared workspace; the call no longer uses one */

/* Geometry of one memory bank (paper notation: L, H_q, H_k, d, G). */
typedef struct stom_oqm_config {
    int32_t n_layers;        /* L                                               */
    int32_t n_q_heads;       /* H_q, a multiple of n_kv_heads                   */
    int32_t n_kv_heads;      /* H_k                                             */
    int32_t head_dim;        /* d: 64, 128 or 256                               */
    int32_t group_tokens;    /* G, tokens per group (frame); 1..64              */
    int32_t capacity_groups; /* groups the bank can hold per layer              */
    int32_t bits;            /* 4 (the paper's setting) or 2 (its ablation)     */
    int32_t kv_dtype;        /* STOM_BF16 | STOM_FP16 | STOM_FP32: type of K, V, Q inputs */
    int32_t score_mode;      /* STOM_SCORE_PER_LAYER | STOM_SCORE_PER_HEAD      */
    int32_t meta_dtype;      /* type the bank keeps s, m and k-bar in: STOM_FP32 (the (s_t, m_t) equation taken
                                in binary32), or STOM_FP16 / STOM_BF16 (half the metadata bytes; see below)   */
} stom_oqm_config;

/*
 * The memory bank M_t (Sec. 3.4): device arrays, all caller-owned, each
 * indexed [layer][group][kv head]... with `capacity_groups` groups per layer.
 *   codes_*   [L][cap][H_k][G][d*bits/8]  uint8: 8/bits codes per byte along
 *             the channel axis, lowest channel in the lowest bits (bits = 4:
 *             two per byte, even channel in the low nibble)
 *   scale_*   [L][cap][H_k][d] meta_dtype: s = (max - min)/15 over the G tokens
 *   zero_*    [L][cap][H_k][d] meta_dtype: m = min over the G tokens
 *   rep_key   [L][cap][H_k][d] meta_dtype: mean of the group's keys (k-bar)
 *   rep_norm2 [L][cap][H_k]    float: squared L2 norm of the STORED k-bar per head
 * With 16-bit metadata (the paper fixes no storage type for the (s_t, m_t) of
 * Sec. 3.4; its experiments run in FP16, Sec. 4.1) the stored offset is the
 * largest 16-bit value <= the channel minimum, the stored scale the smallest
 * 16-bit value >= fl32((max - m)/levels) for that stored m, and the codes are
 * taken against the stored pair: every code stays in range and the
 * reconstruction error stays <= s/2 of the stored s.  k-bar is rounded to
 * nearest-even.  Inputs must then lie inside the 16-bit type's finite range.
 * System-prompt tokens are not part of the bank; they stay in full precision
 * in the caller's active cache.
 */
typedef struct stom_oqm_store {
    uint8_t *codes_k;
    uint8_t *codes_v;
    void *scale_k; /* elements of cfg.meta_dtype, like the next four */
    void *zero_k;
    void *scale_v;
    void *zero_v;
    void *rep_key;
    float *rep_norm2;
} stom_oqm_store;

/* Byte offsets of the eight arrays inside one arena, each 256-byte aligned. */
typedef struct stom_oqm_layout {
    int64_t bytes_total;
    int64_t off_codes_k, off_codes_v;
    int64_t off_scale_k, off_zero_k, off_scale_v, off_zero_v;
    int64_t off_rep_key, off_rep_norm2;
    int64_t bytes_codes;   /* of ONE of codes_k / codes_v   */
    int64_t bytes_meta;    /* of ONE of the four s / m arrays and of rep_key */
    int64_t bytes_norm2;
} stom_oqm_layout;

/* ---- helpers (host only, no CUDA calls) ------------------------------ */

/* Checks `cfg` and fills `out` with the arena layout.  Errors: INVALID_ARG,
 * SHAPE, UNSUPPORTED. */
int32_t stom_oqm_store_layout(const stom_oqm_config *cfg, stom_oqm_layout *out);

/* Points the eight arrays of `out` into `arena` (device memory of at least
 * layout.bytes_total bytes, 256-byte aligned) -- pointer arithmetic only. */
int32_t stom_oqm_store_bind(const stom_oqm_config *cfg, void *arena, stom_oqm_store *out);

/* Appendix, K = min(ceil(B/G), T/G): groups to retrieve for a token budget B
 * when `stored_groups` groups are in the bank. */
int32_t stom_oqm_budget_to_k(int64_t budget_tokens, int32_t group_tokens, int32_t stored_groups);

/* Bytes of scratch stom_oqm_score_groups needs for `layer_count` layers. */
int64_t stom_oqm_score_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count);

const char *stom_status_string(int32_t status);

/* cudaError_t value of the last failed CUDA call made by this library on the
 * calling thread (0 if none). */
int32_t stom_last_cuda_error(void);

/* ---- A1: quantize arriving groups and append them (Sec. 3.4, the Q_4 and
 *      (s_t, m_t) equations; representative key: Sec. 3.4 and appendix
 *      "Layer-wise vision memory") ---------------------------------------
 *
 * For every layer l in [layer_begin, layer_begin+layer_count), frame f in
 * [0, group_count), kv head h and channel c, over the G tokens g of the
 * frame's group:
 *     m = min_g x,  s = (max_g x - m)/15,
 *     code = clamp(rne((x - m)/s), 0, 15)   (binary32, true division;
 *                                            s == 0 -> every code 0)
 * (with cfg->bits == 2, the variant of the paper's ablation table: 3 in place
 * of 15, four codes per byte)
 * for K and for V, and for K also k-bar[c] = mean_g and |k-bar_h|^2.  Results
 * go to bank slot group_begin + f of layer l.  Older groups are never read.
 *
 * K, V (type cfg->kv_dtype): element (l, f, h, tok, c) is at
 *   (l-layer_begin)*stride_layer + f*stride_group + h*stride_head
 *   + tok*stride_token + c,
 * tok = token_idx ? token_idx[f*G + g] : g.
 * K_summary (nullable, same addressing): keys taken before the rotary
 *   embedding, averaged into k-bar instead of K.
 * token_idx (nullable, device, [group_count][G] int32): which of the frame's
 *   tokens_per_frame_in tokens form the group (the pre-LLM selector's keep
 *   list).  Entries outside [0, tokens_per_frame_in) are clamped into range
 *   and STOM_FLAG_BAD_INDEX is set in *dev_flags.
 * dev_flags (nullable, device uint32): OR-ed with STOM_FLAG_* bits.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALIGNMENT, CAPACITY, CUDA.
 */
int32_t stom_oqm_quantize_frame(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                int32_t layer_begin, int32_t layer_count,
                                int32_t group_begin, int32_t group_count,
                                const void *K, const void *V,
                                int64_t stride_layer, int64_t stride_group,
                                int64_t stride_head, int64_t stride_token,
                                const void *K_summary, const int32_t *token_idx,
                                int32_t tokens_per_frame_in, uint32_t *dev_flags, void *stream);

/* ---- A2: question embedding and cosine scores (appendix "Question-guided
 *      single-pass retrieval": the q^(l) equation; Sec. 3.4 sim(q, k-bar)) --
 *
 * q[l][h][c] = mean over the H_q/H_k query heads of kv head h (query head
 * h_q belongs to kv head h_q / (H_q/H_k)) and over the T_q tokens of Q.
 * PER_LAYER: scores[li][t] = <q, k-bar_t> / (max(|q|,1e-12) max(|k-bar_t|,1e-12))
 *   over the flattened H_k*d vector;           scores is [layer_count][n_groups].
 * PER_HEAD:  the same per kv head over d;      scores is [layer_count][H_k][n_groups].
 * Q (type cfg->kv_dtype): element (l, h_q, j, c) at (l-layer_begin)*q_stride_layer
 *   + h_q*q_stride_head + j*q_stride_token + c.
 * workspace: device scratch of stom_oqm_score_workspace_bytes() bytes, 16-byte
 *   aligned; holds the question embeddings between the two kernels.
 * Errors: INVALID_ARG, SHAPE, ALIGNMENT, CAPACITY, WORKSPACE, CUDA.
 */
int32_t stom_oqm_score_groups(const stom_oqm_config *cfg, const stom_oqm_store *store,
                              int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                              const void *Q, int32_t T_q, int64_t q_stride_layer,
                              int64_t q_stride_head, int64_t q_stride_token,
                              float *scores, void *workspace, int64_t workspace_bytes, void *stream);

/* ---- A2 for callers that cannot allocate device memory -----------------
 *
 * (No counterpart in the paper: this is a packaging variant of the call above.)
 *
 * Some hosts of this library have no allocator to offer: an inference server
 * that handed every byte of HBM to its own pool at start-up, a plug-in that is
 * forbidden to call cudaMalloc because that call synchronises the whole device
 * and would stall the other streams of a serving process, or a caller that only
 * holds the tensors it was given.  stom_oqm_score_groups needs a scratch buffer
 * from such a caller; this variant does not.  It computes exactly the same
 * scores with the same kernels, but keeps the question embeddings in a fixed
 * array of STOM_NOALLOC_SCRATCH_BYTES bytes that is part of the library image.
 * Inputs and outputs are still the caller's.
 *
 * Consequences of the built-in array:
 *   - every GPU that loads the library holds the array until the process exits;
 *   - the layer range of one call must fit: layer_count * H_k * (d + 1) * 4
 *     bytes, rounded up to 256, may not exceed STOM_NOALLOC_SCRATCH_BYTES,
 *     otherwise the call returns STOM_ERR_NOALLOC_LIMIT and launches nothing
 *     (score the layers in several calls instead);
 *   - all calls on one GPU share the array.  Calls that may overlap on the GPU
 *     (different streams, no ordering between them) race on it and produce
 *     wrong scores; calls on one stream, or ordered by events, are safe.  The
 *     array keeps the previous call's contents; nothing in it needs clearing,
 *     because each call rewrites every word it later reads;
 *   - the first call on each GPU looks up the array's device address (with that
 *     GPU current) before it launches; make that first call outside of any
 *     stream capture.
 * The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 * Errors: as stom_oqm_score_groups without WORKSPACE, plus NOALLOC_LIMIT, and
 * UNSUPPORTED for a device ordinal of 64 or more.
 */
#define STOM_NOALLOC_SCRATCH_BYTES (512 * 1024)
int32_t stom_oqm_score_groups_noalloc(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                      int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                                      const void *Q, int32_t T_q, int64_t q_stride_layer,
                                      int64_t q_stride_head, int64_t q_stride_token,
                                      float *scores, void *stream);

/* ---- A3: top-K (Sec. 3.4 the TopK equation; appendix: selected indices are
 *      kept in sorted order) ---------------------------------------------
 *
 * For each of `rows` rows of `n` scores (row r starts at scores + r*row_stride):
 * the min(k, n) largest, equal scores resolved towards the lower index, written
 * to idx_out[r][0..] in ASCENDING index order; remaining slots are -1.
 * score_out (nullable, [rows][k]): the selected scores in the same order (0 in
 * unused slots).  n_sel_out (nullable, [rows]): min(k, n).
 * Errors: INVALID_ARG, SHAPE (n above 2^24 is not covered), CUDA.
 */
int32_t stom_oqm_topk(const float *scores, int32_t rows, int32_t n, int64_t row_stride, int32_t k,
                      int32_t *idx_out, float *score_out, int32_t *n_sel_out, void *stream);

/* ---- A4: dequantize the selected groups into the active cache (Sec. 3.4,
 *      the Q_4^{-1} and KV_active equations; appendix "Cache reconstruction
 *      for decoding") -----------------------------------------------------
 *
 * idx (device int32): PER_LAYER [layer_count][k]; PER_HEAD [layer_count][H_k][k].
 * For slot j holding group t >= 0, every kv head h, token g, channel c:
 *   out[l][h][token_offset + j*G + g][c] = round_to_out_dtype(fmaf(code, s, m))
 * for K into k_active and V into v_active; element (l, h, tok, c) is at
 * (l-layer_begin)*stride_layer + h*stride_head + tok*stride_token + c.
 * Slots with idx == -1 are left untouched; idx < -1 or >= n_groups is skipped
 * and flagged in *dev_flags (nullable).  token_offset is the number of
 * system-prompt tokens that precede the visual groups in the active cache.
 * out_dtype: STOM_BF16 or STOM_FP16.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALIGNMENT, CAPACITY, CUDA.
 */
int32_t stom_oqm_dequant_gather(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                int32_t layer_begin, int32_t layer_count,
                                const int32_t *idx, int32_t k, int32_t n_groups,
                                void *k_active, void *v_active, int32_t out_dtype,
                                int64_t stride_layer, int64_t stride_head, int64_t stride_token,
                                int32_t token_offset, uint32_t *dev_flags, void *stream);

/* ---- A2+A3+A4 in one call (Sec. 3.4: retrieval then selective
 *      reconstruction, once per question) ---------------------------------
 * Same arguments as the three calls above; scores, idx are caller buffers that
 * receive the intermediate results ([rows][n_groups] and [rows][k]).
 * workspace: at least stom_oqm_score_workspace_bytes() bytes, 16-byte aligned.
 * With stom_oqm_retrieve_workspace_bytes() bytes, 256-byte aligned, the
 * selection runs in two levels (every block pre-selects in its own run of
 * groups), which shortens the call; the results are the same.
 */
int64_t stom_oqm_retrieve_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count,
                                          int32_t n_groups, int32_t k);
int32_t stom_oqm_retrieve(const stom_oqm_config *cfg, const stom_oqm_store *store,
                          int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                          const void *Q, int32_t T_q, int64_t q_stride_layer,
                          int64_t q_stride_head, int64_t q_stride_token,
                          int32_t k, float *scores, int32_t *idx,
                          void *k_active, void *v_active, int32_t out_dtype,
                          int64_t stride_layer, int64_t stride_head, int64_t stride_token,
                          int32_t token_offset, void *workspace, int64_t workspace_bytes,
                          uint32_t *dev_flags, void *stream);

/* ---- A5: decode attention over [system tokens || selected groups] without
 *      materialising the cache (Sec. 3.4: decoding attends to the bounded
 *      active kv; appendix "Cache reconstruction for decoding": the per-layer
 *      indices are reused for every decode step) ---------------------------
 *
 * For every layer of the range and every query head h_q (kv head h = h_q /
 * (H_q/H_k)):  out[l][h_q][:] = softmax_t(softmax_scale * <q[l][h_q], K_t>) V_t
 * over the tokens t of  [the sys_len system tokens of (l, h)] followed by [the
 * G tokens of every selected group idx[..][j] >= 0, j < k], where a group's K
 * and V rows are code * s + m of the bank (not rounded to a 16-bit type on the
 * way).  Accumulation is binary32; the output is rounded once to cache_dtype.
 * Both contractions run on the tensor cores with the raw codes as one operand
 * (exact) and q*s, respectively the softmax weights, as the other, carried as
 * a high and a low 16-bit part (16 significant bits); the affine terms are
 * added in binary32.
 * idx: as for stom_oqm_dequant_gather (PER_LAYER [layer_count][k]; PER_HEAD
 *   [layer_count][H_k][k]); -1 entries are skipped, other out-of-range entries
 *   are skipped and flagged.  k may be 0 if sys_len > 0.
 * q_dec (cfg->kv_dtype): element (l, h_q, c) at (l-layer_begin)*q_stride_layer
 *   + h_q*q_stride_head + c; 4-byte aligned, both strides a multiple of 4 bytes.
 * k_sys, v_sys (cache_dtype = STOM_BF16 | STOM_FP16; may be NULL if sys_len == 0):
 *   element (l, h, tok, c) at (l-layer_begin)*sys_stride_layer + h*sys_stride_head
 *   + tok*sys_stride_token + c -- the first sys_len tokens of the active cache.
 * out (cache_dtype): element (l, h_q, c) at (l-layer_begin)*out_stride_layer +
 *   h_q*out_stride_head + c.
 * workspace, workspace_bytes: not used.  The blocks that share a (layer, kv
 *   head) combine their partial results through the shared memory of a
 *   thread-block cluster, so the call keeps nothing in global memory between
 *   or during launches; the two arguments remain so that callers written for
 *   the earlier form of the call (which took a cleared scratch buffer) keep
 *   working, and may be NULL / 0.  stom_oqm_attend_workspace_bytes() returns a
 *   small constant.  STOM_FLAG_DIRTY_WORKSPACE is no longer raised.
 * A bulk copy into shared memory that has not landed after 2 s ends the block
 * that waits for it: STOM_FLAG_TIMEOUT is set in dev_flags and the output rows
 * of that (layer, kv head) are void.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALIGNMENT, CAPACITY, CUDA.
 */
int64_t stom_oqm_attend_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count, int32_t k,
                                        int32_t sys_len);
int32_t stom_oqm_attend(const stom_oqm_config *cfg, const stom_oqm_store *store,
                        int32_t layer_begin, int32_t layer_count,
                        const int32_t *idx, int32_t k, int32_t n_groups,
                        const void *q_dec, int64_t q_stride_layer, int64_t q_stride_head,
                        const void *k_sys, const void *v_sys, int32_t cache_dtype,
                        int64_t sys_stride_layer, int64_t sys_stride_head, int64_t sys_stride_token,
                        int32_t sys_len, float softmax_scale,
                        void *out, int64_t out_stride_layer, int64_t out_stride_head,
                        void *workspace, int64_t workspace_bytes, uint32_t *dev_flags, void *stream);

/* ---- the same path driven from HOST memory -----------------------------
 * These two calls take HOST input/output buffers (pinned memory makes the
 * copies asynchronous), stage them through caller-provided DEVICE scratch with
 * cudaMemcpyAsync on `stream`, and run the kernels of A1 resp. A2-A4 above
 * (same passages of the paper).  They return without synchronising: results
 * in host memory are valid after the caller synchronises the stream.
 */

/* Device scratch bytes stom_oqm_quantize_frame_host needs. */
int64_t stom_oqm_quantize_host_scratch_bytes(const stom_oqm_config *cfg, int32_t layer_count,
                                             int32_t group_count);

/* A1 from host memory.  K_host, V_host: compact [layer_count][group_count][H_k][G][d]
 * arrays of cfg->kv_dtype on the HOST.  scratch: DEVICE, 16-byte aligned.
 * Errors: as stom_oqm_quantize_frame, plus WORKSPACE. */
int32_t stom_oqm_quantize_frame_host(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                     int32_t layer_begin, int32_t layer_count,
                                     int32_t group_begin, int32_t group_count,
                                     const void *K_host, const void *V_host,
                                     void *scratch, int64_t scratch_bytes, uint32_t *dev_flags,
                                     void *stream);

/* Device scratch bytes stom_oqm_retrieve_host needs. */
int64_t stom_oqm_retrieve_host_scratch_bytes(const stom_oqm_config *cfg, int32_t layer_count,
                                             int32_t n_groups, int32_t T_q, int32_t k, int32_t out_dtype);

/* A2+A3+A4 from host memory.  Q_host: compact [layer_count][H_q][T_q][d] of
 * cfg->kv_dtype on the HOST.  idx_host: HOST [rows][k] int32 (rows as in
 * stom_oqm_topk).  k_active_host, v_active_host: HOST compact
 * [layer_count][H_k][k*G][d] of out_dtype, both given or both NULL (NULL: the
 * reconstructed cache stays in scratch on the device and is not copied back).
 * When fewer than k groups are stored, the token slots behind the last
 * selected group (those of idx == -1) come back as zeros.
 * scratch: DEVICE, 256-byte aligned.
 * Errors: as the three device calls, plus WORKSPACE. */
int32_t stom_oqm_retrieve_host(const stom_oqm_config *cfg, const stom_oqm_store *store,
                               int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                               const void *Q_host, int32_t T_q, int32_t k,
                               int32_t *idx_host, void *k_active_host, void *v_active_host,
                               int32_t out_dtype, void *scratch, int64_t scratch_bytes,
                               uint32_t *dev_flags, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* STOM_OQM_H */
