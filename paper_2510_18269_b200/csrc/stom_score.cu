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

#include "stom_internal.cuh"

namespace stom {

struct ScoreParams {
    const void *Q;
    int64_t ql, qh, qt;  // element strides of Q: layer, head, token
    const float *rep_key, *rep_norm2;
    float *qemb;    // workspace: [layer_count][H][d]
    float *qnorm2;  // workspace: [layer_count][H]
    float *scores;
    BankGeom g;
    int32_t layer_begin, layer_count, n_groups, T_q, rep, per_head;
};

// grid (H, layer_count), block d threads: thread c owns channel c of kv head h
template <typename T>
__global__ void query_embed_kernel(const ScoreParams p) {
    const int h = blockIdx.x, li = blockIdx.y, c = threadIdx.x, d = p.g.d;
    const T *q = reinterpret_cast<const T *>(p.Q) + (int64_t)li * p.ql + c;
    float acc = 0.0f;
    for (int r = 0; r < p.rep; ++r) {
        const T *qh = q + (int64_t)(h * p.rep + r) * p.qh;
        float part = 0.0f;
        for (int j = 0; j < p.T_q; ++j) part += (float)qh[(int64_t)j * p.qt];
        acc += part;
    }
    const float v = acc / (float)(p.rep * p.T_q);
    p.qemb[((int64_t)li * p.g.H + h) * d + c] = v;
    // |q_h|^2 by block reduction
    __shared__ float red[8];
    float sq = v * v;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((c & 31) == 0) red[c >> 5] = sq;
    __syncthreads();
    if (c == 0) {
        float tot = 0.0f;
        for (int w = 0; w < (d >> 5); ++w) tot += red[w];
        p.qnorm2[(int64_t)li * p.g.H + h] = tot;
    }
}

constexpr int kScoreWarps = 8;
constexpr int kGroupsPerWarp = 4;  // groups a warp scores one after the other per block

// grid (ceil(n_groups / (kScoreWarps*kGroupsPerWarp)), layer_count)
__global__ void __launch_bounds__(kScoreWarps * 32) score_kernel(const ScoreParams p) {
    extern __shared__ __align__(16) float sq[];  // q of this layer: H*d floats, then H norms
    const int li = blockIdx.y, H = p.g.H, d = p.g.d, HD = H * d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < HD; i += blockDim.x) sq[i] = p.qemb[(int64_t)li * HD + i];
    float *qn = sq + HD;
    if (threadIdx.x < H) qn[threadIdx.x] = p.qnorm2[(int64_t)li * H + threadIdx.x];
    __syncthreads();

    const int l = p.layer_begin + li;
    const float eps = 1e-12f;
    const int t0 = (blockIdx.x * kScoreWarps + warp) * kGroupsPerWarp;
#pragma unroll 1
    for (int u = 0; u < kGroupsPerWarp; ++u) {
        const int t = t0 + u;
        if (t >= p.n_groups) break;
        const int64_t slot = bank_slot(p.g, l, t, 0);
        const float4 *kb = reinterpret_cast<const float4 *>(p.rep_key + slot * d);
        if (!p.per_head) {
            float dot = 0.0f;
            for (int i = lane; i < HD / 4; i += 32) {
                const float4 a = __ldg(kb + i);
                const float4 b = reinterpret_cast<const float4 *>(sq)[i];
                dot = fmaf(a.x, b.x, dot);
                dot = fmaf(a.y, b.y, dot);
                dot = fmaf(a.z, b.z, dot);
                dot = fmaf(a.w, b.w, dot);
            }
            float kn = 0.0f, qq = 0.0f;
            for (int hh = lane; hh < H; hh += 32) {
                kn += __ldg(p.rep_norm2 + slot + hh);
                qq += qn[hh];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                dot += __shfl_xor_sync(0xffffffffu, dot, o);
                kn += __shfl_xor_sync(0xffffffffu, kn, o);
                qq += __shfl_xor_sync(0xffffffffu, qq, o);
            }
            if (lane == 0)
                p.scores[(int64_t)li * p.n_groups + t] = dot / (fmaxf(sqrtf(qq), eps) * fmaxf(sqrtf(kn), eps));
        } else {
            for (int hh = 0; hh < H; ++hh) {
                float dot = 0.0f;
                for (int i = lane; i < d / 4; i += 32) {
                    const float4 a = __ldg(kb + hh * (d / 4) + i);
                    const float4 b = reinterpret_cast<const float4 *>(sq)[hh * (d / 4) + i];
                    dot = fmaf(a.x, b.x, dot);
                    dot = fmaf(a.y, b.y, dot);
                    dot = fmaf(a.z, b.z, dot);
                    dot = fmaf(a.w, b.w, dot);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                if (lane == 0) {
                    const float kn = __ldg(p.rep_norm2 + slot + hh);
                    p.scores[((int64_t)li * H + hh) * p.n_groups + t] =
                        dot / (fmaxf(sqrtf(qn[hh]), eps) * fmaxf(sqrtf(kn), eps));
                }
            }
        }
    }
}

}  // namespace stom

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
    if (reinterpret_cast<uintptr_t>(Q) % elem_bytes(cfg->kv_dtype) || (reinterpret_cast<uintptr_t>(scores) & 3u))
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
    case STOM_BF16: query_embed_kernel<__nv_bfloat16><<<g1, cfg->head_dim, 0, s>>>(p); break;
    case STOM_FP16: query_embed_kernel<__half><<<g1, cfg->head_dim, 0, s>>>(p); break;
    default: query_embed_kernel<float><<<g1, cfg->head_dim, 0, s>>>(p); break;
    }
    if ((rc = finish_launch())) return rc;

    const int per_block = kScoreWarps * kGroupsPerWarp;
    dim3 g2((n_groups + per_block - 1) / per_block, layer_count);
    const size_t smem = (size_t)cfg->n_kv_heads * (cfg->head_dim + 1) * sizeof(float);
    score_kernel<<<g2, kScoreWarps * 32, smem, s>>>(p);
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
