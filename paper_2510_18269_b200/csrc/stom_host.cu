// Entry points that take HOST buffers: they copy the inputs to caller-provided
// device scratch, run the same kernels as the device-pointer entry points, and
// copy the results back.  They exist so that a caller (and the end-to-end
// measurement) can drive the path from host memory through the C ABI.  All
// copies are cudaMemcpyAsync on the caller's stream; pinned host memory makes
// them truly asynchronous.  Nothing is allocated here.
#include "stom_internal.cuh"

using namespace stom;

static int64_t up256(int64_t x) { return (x + 255) / 256 * 256; }

static int32_t copy_async(void *dst, const void *src, int64_t bytes, cudaMemcpyKind kind, cudaStream_t s) {
    cudaError_t e = cudaMemcpyAsync(dst, src, (size_t)bytes, kind, s);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    return STOM_OK;
}

extern "C" int64_t stom_oqm_quantize_host_scratch_bytes(const stom_oqm_config *cfg, int32_t layer_count,
                                                        int32_t group_count) {
    if (check_config(cfg) || layer_count < 0 || group_count < 0) return STOM_ERR_INVALID_ARG;
    const int64_t one = (int64_t)layer_count * group_count * cfg->n_kv_heads * cfg->group_tokens * cfg->head_dim *
                        elem_bytes(cfg->kv_dtype);
    return 2 * up256(one);
}

extern "C" int32_t stom_oqm_quantize_frame_host(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                                int32_t layer_begin, int32_t layer_count,
                                                int32_t group_begin, int32_t group_count,
                                                const void *K_host, const void *V_host,
                                                void *scratch, int64_t scratch_bytes, uint32_t *dev_flags,
                                                void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if (!K_host || !V_host) return STOM_ERR_INVALID_ARG;
    if (layer_count < 0 || group_count < 0) return STOM_ERR_INVALID_ARG;
    const int64_t need = stom_oqm_quantize_host_scratch_bytes(cfg, layer_count, group_count);
    if (!scratch || !aligned16(scratch) || scratch_bytes < need) return STOM_ERR_WORKSPACE;
    if (layer_count == 0 || group_count == 0) return STOM_OK;
    const int64_t H = cfg->n_kv_heads, G = cfg->group_tokens, d = cfg->head_dim;
    const int64_t one = (int64_t)layer_count * group_count * H * G * d * elem_bytes(cfg->kv_dtype);
    uint8_t *dK = static_cast<uint8_t *>(scratch), *dV = dK + up256(one);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((rc = copy_async(dK, K_host, one, cudaMemcpyHostToDevice, s))) return rc;
    if ((rc = copy_async(dV, V_host, one, cudaMemcpyHostToDevice, s))) return rc;
    return stom_oqm_quantize_frame(cfg, store, layer_begin, layer_count, group_begin, group_count, dK, dV,
                                   (int64_t)group_count * H * G * d, H * G * d, G * d, d, nullptr, nullptr, 0,
                                   dev_flags, stream);
}

namespace {
struct RetrieveScratch {
    int64_t off_q, off_scores, off_idx, off_ws, off_ka, off_va, total;
    int64_t bytes_q, bytes_idx, bytes_act;
};
RetrieveScratch retrieve_scratch(const stom_oqm_config *cfg, int32_t layer_count, int32_t n_groups, int32_t T_q,
                                 int32_t k, int32_t out_dtype) {
    RetrieveScratch r;
    const int64_t rows = (int64_t)layer_count * (cfg->score_mode == STOM_SCORE_PER_HEAD ? cfg->n_kv_heads : 1);
    r.bytes_q = (int64_t)layer_count * cfg->n_q_heads * T_q * cfg->head_dim * elem_bytes(cfg->kv_dtype);
    r.bytes_idx = rows * k * 4;
    r.bytes_act = (int64_t)layer_count * cfg->n_kv_heads * k * cfg->group_tokens * cfg->head_dim * elem_bytes(out_dtype);
    int64_t off = 0;
    r.off_q = off; off += up256(r.bytes_q);
    r.off_scores = off; off += up256(rows * (int64_t)n_groups * 4);
    r.off_idx = off; off += up256(r.bytes_idx);
    r.off_ws = off; off += up256(stom_oqm_retrieve_workspace_bytes(cfg, layer_count, n_groups, k));
    r.off_ka = off; off += up256(r.bytes_act);
    r.off_va = off; off += up256(r.bytes_act);
    r.total = off;
    return r;
}
}  // namespace

extern "C" int64_t stom_oqm_retrieve_host_scratch_bytes(const stom_oqm_config *cfg, int32_t layer_count,
                                                        int32_t n_groups, int32_t T_q, int32_t k, int32_t out_dtype) {
    if (check_config(cfg) || layer_count < 0 || n_groups < 0 || T_q < 1 || k < 1) return STOM_ERR_INVALID_ARG;
    if (out_dtype != STOM_BF16 && out_dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    return retrieve_scratch(cfg, layer_count, n_groups, T_q, k, out_dtype).total;
}

extern "C" int32_t stom_oqm_retrieve_host(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                          int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                                          const void *Q_host, int32_t T_q, int32_t k,
                                          int32_t *idx_host, void *k_active_host, void *v_active_host,
                                          int32_t out_dtype, void *scratch, int64_t scratch_bytes,
                                          uint32_t *dev_flags, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if (!Q_host || !idx_host || layer_count < 0 || n_groups < 0 || T_q < 1 || k < 1) return STOM_ERR_INVALID_ARG;
    if ((k_active_host == nullptr) != (v_active_host == nullptr)) return STOM_ERR_INVALID_ARG;
    if (out_dtype != STOM_BF16 && out_dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    const RetrieveScratch r = retrieve_scratch(cfg, layer_count, n_groups, T_q, k, out_dtype);
    if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255u) || scratch_bytes < r.total) return STOM_ERR_WORKSPACE;
    if (layer_count == 0) return STOM_OK;
    uint8_t *b = static_cast<uint8_t *>(scratch);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t d = cfg->head_dim, S = (int64_t)k * cfg->group_tokens;
    if ((rc = copy_async(b + r.off_q, Q_host, r.bytes_q, cudaMemcpyHostToDevice, s))) return rc;
    if (n_groups < k && k_active_host) {
        // slots behind the last stored group are not written by the gather: hand back zeros, not stale scratch
        cudaError_t e = cudaMemsetAsync(b + r.off_ka, 0, (size_t)(r.off_va + up256(r.bytes_act) - r.off_ka), s);
        if (e != cudaSuccess) {
            set_last_cuda_error(e);
            return STOM_ERR_CUDA;
        }
    }
    rc = stom_oqm_retrieve(cfg, store, layer_begin, layer_count, n_groups, b + r.off_q, T_q,
                           (int64_t)cfg->n_q_heads * T_q * d, (int64_t)T_q * d, d, k,
                           reinterpret_cast<float *>(b + r.off_scores), reinterpret_cast<int32_t *>(b + r.off_idx),
                           b + r.off_ka, b + r.off_va, out_dtype, (int64_t)cfg->n_kv_heads * S * d, S * d, d, 0,
                           b + r.off_ws, up256(stom_oqm_retrieve_workspace_bytes(cfg, layer_count, n_groups, k)), dev_flags, stream);
    if (rc) return rc;
    if ((rc = copy_async(idx_host, b + r.off_idx, r.bytes_idx, cudaMemcpyDeviceToHost, s))) return rc;
    if (k_active_host) {
        if ((rc = copy_async(k_active_host, b + r.off_ka, r.bytes_act, cudaMemcpyDeviceToHost, s))) return rc;
        if ((rc = copy_async(v_active_host, b + r.off_va, r.bytes_act, cudaMemcpyDeviceToHost, s))) return rc;
    }
    return STOM_OK;
}
