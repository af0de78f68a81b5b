// A2: question embedding and cosine scores over the representative keys
// (paper appendix "Question-guided single-pass retrieval": average the query
// heads of each GQA block, average over the question tokens, flatten,
// L2-normalise, cosine; Sec. 3.4 sim(q, k-bar_i)).
//
// The T_q question tokens are averaged away BEFORE the similarity, so per
// layer this is a matrix-vector product over the [T][H_k*d] bank of
// representative keys: memory-bound streaming, no tensor cores.
//   kernel 1: q[l][h][:] and |q_h|^2 -> workspace            (tiny)
//   kernel 2: one warp per stored group, q held in shared memory, 16-byte
//             loads of k-bar, warp-shuffle reduction, stored |k-bar_h|^2
//             reused for the norm.
#include <mutex>

#include "stom_score.cuh"

using namespace stom;

extern "C" int64_t stom_oqm_score_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count) {
    if (check_config(cfg) || layer_count < 0) return STOM_ERR_INVALID_ARG;
    // question embeddings [layer_count][H][d] then their squared norms [layer_count][H]
    const int64_t n = (int64_t)layer_count * cfg->n_kv_heads * (cfg->head_dim + 1) * 4;
    return (n + 255) / 256 * 256;
}

extern "C" int32_t stom_oqm_score_groups(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                         int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                                         const void *Q, int32_t T_q, int64_t q_stride_layer,
                                         int64_t q_stride_head, int64_t q_stride_token,
                                         float *scores, void *workspace, int64_t workspace_bytes, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if ((rc = check_store(store))) return rc;
    if ((rc = check_layers(cfg, layer_begin, layer_count))) return rc;
    if (!Q || !scores || T_q < 1 || n_groups < 0) return STOM_ERR_INVALID_ARG;
    if (n_groups > cfg->capacity_groups) return STOM_ERR_CAPACITY;
    if (q_stride_layer < 0 || q_stride_head < 0 || q_stride_token < 0) return STOM_ERR_INVALID_ARG;
    if (!workspace || !aligned16(workspace) || workspace_bytes < stom_oqm_score_workspace_bytes(cfg, layer_count))
        return STOM_ERR_WORKSPACE;
    if (!aligned16(Q) || (reinterpret_cast<uintptr_t>(scores) & 3u)) return STOM_ERR_ALIGNMENT;
    if (!stride_ok(q_stride_layer, cfg->kv_dtype) || !stride_ok(q_stride_head, cfg->kv_dtype) ||
        !stride_ok(q_stride_token, cfg->kv_dtype))
        return STOM_ERR_ALIGNMENT;
    if (layer_count == 0 || n_groups == 0) return STOM_OK;

    ScoreParams p;
    p.Q = Q; p.ql = q_stride_layer; p.qh = q_stride_head; p.qt = q_stride_token;
    p.rep_key = store->rep_key; p.rep_norm2 = store->rep_norm2;
    p.qemb = static_cast<float *>(workspace);
    p.qnorm2 = p.qemb + (int64_t)layer_count * cfg->n_kv_heads * cfg->head_dim;
    p.scores = scores;
    p.g = bank_geom(cfg);
    p.layer_begin = layer_begin; p.layer_count = layer_count; p.n_groups = n_groups; p.T_q = T_q;
    p.rep = cfg->n_q_heads / cfg->n_kv_heads;
    p.per_head = cfg->score_mode == STOM_SCORE_PER_HEAD;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    dim3 g1(cfg->n_kv_heads, layer_count);
    switch (cfg->kv_dtype) {
    case STOM_BF16: query_embed_kernel<__nv_bfloat16><<<g1, kEmbedThreads, 0, s>>>(p); break;
    case STOM_FP16: query_embed_kernel<__half><<<g1, kEmbedThreads, 0, s>>>(p); break;
    default: query_embed_kernel<float><<<g1, kEmbedThreads, 0, s>>>(p); break;
    }
    if ((rc = finish_launch())) return rc;

    // about two blocks per SM over the whole grid, each with a long contiguous run of groups (at least 32): a block's
    // first loads and its last reduction are paid once per run.  The kernel is launched so that its blocks may be
    // scheduled under the tail of the embedding kernel; it waits for that kernel before it reads the embeddings.
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    int chunks = (2 * sms) / layer_count;
    if (chunks > (n_groups + 31) / 32) chunks = (n_groups + 31) / 32;
    if (chunks < 1) chunks = 1;
    p.groups_per_block = (n_groups + chunks - 1) / chunks;
    dim3 g2((n_groups + p.groups_per_block - 1) / p.groups_per_block, layer_count);
    const size_t smem = (size_t)cfg->n_kv_heads * (cfg->head_dim + 1) * sizeof(float);
    const int HD = cfg->n_kv_heads * cfg->head_dim;
    const bool fast = !p.per_head && cfg->n_kv_heads <= 32;
    cudaError_t le = cudaSuccess;
#define STOM_SCORE_LAUNCH(KT_)                                                                       \
    switch (score_fast_v4(HD, fast, cfg->meta_dtype)) {                                             \
    case 4: le = launch_after_producer(score_kernel<4, KT_>, g2, dim3(kScoreWarps * 32), smem, s, p); break; /* 4 kv heads x 128 */ \
    case 8: le = launch_after_producer(score_kernel<8, KT_>, g2, dim3(kScoreWarps * 32), smem, s, p); break; /* 8 kv heads x 128 */ \
    case 2: le = launch_after_producer(score_kernel<2, KT_>, g2, dim3(kScoreWarps * 32), smem, s, p); break;                      \
    case 1:                                                                                         \
        if constexpr (sizeof(KT_) == 4) {                                                           \
            le = launch_after_producer(score_kernel<1, KT_>, g2, dim3(kScoreWarps * 32), smem, s, p);                             \
            break;                                                                                  \
        }                                                                                           \
    default: le = launch_after_producer(score_kernel<0, KT_>, g2, dim3(kScoreWarps * 32), smem, s, p); break;                     \
    }
    switch (cfg->meta_dtype) {
    case STOM_BF16: STOM_SCORE_LAUNCH(__nv_bfloat16) break;
    case STOM_FP16: STOM_SCORE_LAUNCH(__half) break;
    default: STOM_SCORE_LAUNCH(float) break;
    }
#undef STOM_SCORE_LAUNCH
    if (le != cudaSuccess) {
        set_last_cuda_error(le);
        return STOM_ERR_CUDA;
    }
    return finish_launch();
}

// ---------------------------------------------------------------------------
// Scoring for callers that must not touch the device allocator.
//
// The question embeddings that pass from the first scoring kernel to the second
// live in an array that is part of the library image instead of in caller
// scratch.  The array exists once per GPU that loads the library and is shared
// by every call on that GPU.
// ---------------------------------------------------------------------------

static __device__ __align__(256) unsigned char g_score_scratch[STOM_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void *g_scratch_addr[kMaxDevices];  // device address of g_score_scratch on each GPU, filled on first use
}  // namespace

extern "C" int32_t stom_oqm_score_groups_noalloc(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                                 int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                                                 const void *Q, int32_t T_q, int64_t q_stride_layer,
                                                 int64_t q_stride_head, int64_t q_stride_token,
                                                 float *scores, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if ((rc = check_layers(cfg, layer_begin, layer_count))) return rc;
    const int64_t need = stom_oqm_score_workspace_bytes(cfg, layer_count);
    if (need < 0) return STOM_ERR_INVALID_ARG;
    if (need > (int64_t)STOM_NOALLOC_SCRATCH_BYTES) return STOM_ERR_NOALLOC_LIMIT;

    // The symbol's name is only a host-side handle; the kernels need its address on the current GPU.
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    if (dev < 0 || dev >= kMaxDevices) return STOM_ERR_UNSUPPORTED;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_score_scratch);
            if (e != cudaSuccess || !p) {
                set_last_cuda_error(e);
                return STOM_ERR_CUDA;
            }
            g_scratch_addr[dev] = p;
        }
        scratch = g_scratch_addr[dev];
    }
    // Every word of the scratch that the second kernel reads is written by the first kernel of the
    // same call, so nothing has to be cleared between calls.
    return stom_oqm_score_groups(cfg, store, layer_begin, layer_count, n_groups, Q, T_q, q_stride_layer,
                                 q_stride_head, q_stride_token, scores, scratch, STOM_NOALLOC_SCRATCH_BYTES, stream);
}
