// Host-only part of the C ABI: geometry checks, arena layout, status strings,
// and the error bookkeeping.
#include "stom_internal.cuh"

namespace stom {

static thread_local int32_t g_last_cuda_error = 0;

void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int32_t)e; }

int32_t check_config(const stom_oqm_config *c) {
    if (!c) return STOM_ERR_INVALID_ARG;
    if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->capacity_groups < 1) return STOM_ERR_INVALID_ARG;
    if (c->n_q_heads % c->n_kv_heads) return STOM_ERR_SHAPE;
    if (c->bits != 4 && c->bits != 2) return STOM_ERR_UNSUPPORTED;
    if (c->kv_dtype != STOM_BF16 && c->kv_dtype != STOM_FP16 && c->kv_dtype != STOM_FP32) return STOM_ERR_UNSUPPORTED;
    if (c->score_mode != STOM_SCORE_PER_LAYER && c->score_mode != STOM_SCORE_PER_HEAD) return STOM_ERR_UNSUPPORTED;
    if (c->meta_dtype != STOM_BF16 && c->meta_dtype != STOM_FP16 && c->meta_dtype != STOM_FP32) return STOM_ERR_UNSUPPORTED;
    if (c->head_dim != 64 && c->head_dim != 128 && c->head_dim != 256) return STOM_ERR_SHAPE;
    if (c->group_tokens < 1 || c->group_tokens > 64) return STOM_ERR_SHAPE;
    // one (group, head) block of codes must keep 16-byte alignment for vector stores
    if (((int64_t)c->group_tokens * c->head_dim * c->bits / 8) % 16) return STOM_ERR_SHAPE;
    return STOM_OK;
}

int32_t check_store(const stom_oqm_store *s) {
    if (!s) return STOM_ERR_INVALID_ARG;
    const void *p[8] = {s->codes_k, s->codes_v, s->scale_k, s->zero_k, s->scale_v, s->zero_v, s->rep_key, s->rep_norm2};
    for (int i = 0; i < 8; ++i) {
        if (!p[i]) return STOM_ERR_INVALID_ARG;
        if (!aligned16(p[i])) return STOM_ERR_ALIGNMENT;
    }
    return STOM_OK;
}

int32_t check_layers(const stom_oqm_config *c, int32_t layer_begin, int32_t layer_count) {
    if (layer_begin < 0 || layer_count < 0) return STOM_ERR_INVALID_ARG;
    if ((int64_t)layer_begin + layer_count > c->n_layers) return STOM_ERR_INVALID_ARG;
    return STOM_OK;
}

}  // namespace stom

using namespace stom;

static int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

extern "C" int32_t stom_oqm_store_layout(const stom_oqm_config *cfg, stom_oqm_layout *out) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if (!out) return STOM_ERR_INVALID_ARG;
    const int64_t slots = (int64_t)cfg->n_layers * cfg->capacity_groups * cfg->n_kv_heads;
    out->bytes_codes = slots * cfg->group_tokens * (cfg->head_dim * cfg->bits / 8);
    out->bytes_meta = slots * cfg->head_dim * elem_bytes(cfg->meta_dtype);
    out->bytes_norm2 = slots * 4;
    int64_t off = 0;
    out->off_codes_k = off; off = round_up(off + out->bytes_codes, 256);
    out->off_codes_v = off; off = round_up(off + out->bytes_codes, 256);
    out->off_scale_k = off; off = round_up(off + out->bytes_meta, 256);
    out->off_zero_k = off;  off = round_up(off + out->bytes_meta, 256);
    out->off_scale_v = off; off = round_up(off + out->bytes_meta, 256);
    out->off_zero_v = off;  off = round_up(off + out->bytes_meta, 256);
    out->off_rep_key = off; off = round_up(off + out->bytes_meta, 256);
    out->off_rep_norm2 = off; off = round_up(off + out->bytes_norm2, 256);
    out->bytes_total = off;
    return STOM_OK;
}

extern "C" int32_t stom_oqm_store_bind(const stom_oqm_config *cfg, void *arena, stom_oqm_store *out) {
    stom_oqm_layout lay;
    int32_t rc = stom_oqm_store_layout(cfg, &lay);
    if (rc) return rc;
    if (!arena || !out) return STOM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(arena) & 255u) return STOM_ERR_ALIGNMENT;
    uint8_t *b = static_cast<uint8_t *>(arena);
    out->codes_k = b + lay.off_codes_k;
    out->codes_v = b + lay.off_codes_v;
    out->scale_k = b + lay.off_scale_k;
    out->zero_k = b + lay.off_zero_k;
    out->scale_v = b + lay.off_scale_v;
    out->zero_v = b + lay.off_zero_v;
    out->rep_key = b + lay.off_rep_key;
    out->rep_norm2 = reinterpret_cast<float *>(b + lay.off_rep_norm2);
    return STOM_OK;
}

extern "C" int32_t stom_oqm_budget_to_k(int64_t budget_tokens, int32_t group_tokens, int32_t stored_groups) {
    if (budget_tokens < 0 || group_tokens < 1 || stored_groups < 0) return STOM_ERR_INVALID_ARG;
    int64_t k = (budget_tokens + group_tokens - 1) / group_tokens;
    return (int32_t)(k < stored_groups ? k : stored_groups);
}

extern "C" const char *stom_status_string(int32_t s) {
    switch (s) {
    case STOM_OK: return "ok";
    case STOM_ERR_INVALID_ARG: return "invalid argument (null pointer, negative count or bad range)";
    case STOM_ERR_SHAPE: return "geometry not covered (head_dim must be 64/128/256, 1 <= group_tokens <= 64, H_q a multiple of H_k)";
    case STOM_ERR_ALIGNMENT: return "pointer or stride breaks the 16-byte alignment rule";
    case STOM_ERR_CAPACITY: return "group range exceeds capacity_groups";
    case STOM_ERR_INDEX: return "index out of range";
    case STOM_ERR_UNSUPPORTED: return "unsupported bits, dtype or mode";
    case STOM_ERR_CUDA: return "CUDA launch failed (see stom_last_cuda_error)";
    case STOM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case STOM_ERR_NOALLOC_LIMIT: return "request needs more scratch than the library's built-in array holds; split the layer range";
    default: return "unknown status";
    }
}

extern "C" int32_t stom_last_cuda_error(void) { return g_last_cuda_error; }
