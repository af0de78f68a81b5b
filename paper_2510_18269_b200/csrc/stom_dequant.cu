// A4: dequantize the selected groups into the bounded active cache (paper
// Sec. 3.4: Q_4^{-1} = depack * s + m and KV_active = union of the selected
// groups; appendix "Cache reconstruction for decoding").
//
// One warp owns one item = (layer, selected slot j, kv head, K|V): G rows of
// d/2 packed bytes in, G rows of d 16-bit values out.  A lane owns 8 adjacent
// channels: it keeps their 8 (s, m) pairs in registers for the whole group,
// reads 4 bytes of codes per row and writes one 16-byte vector per row, so a
// warp's store instruction covers 512 contiguous bytes of the active cache.
// Output bytes are 3/4 of the traffic; code words of a whole group are
// requested before the first one is used.
#include "stom_internal.cuh"

namespace stom {

constexpr int kDqWarps = 4;

struct DequantParams {
    const int32_t *idx;
    const uint8_t *codes_k, *codes_v;
    const float *scale_k, *zero_k, *scale_v, *zero_v;
    void *ka, *va;
    int64_t sl, sh, st;  // element strides of the active cache: layer, head, token
    BankGeom g;
    int32_t layer_begin, k, n_groups, token_offset, per_head;
    uint32_t *flags;
    int64_t n_items;
};

template <typename OT>
__global__ void __launch_bounds__(kDqWarps * 32) dequant_gather_kernel(const DequantParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t item = (int64_t)blockIdx.x * kDqWarps + warp;
    if (item >= p.n_items) return;
    const int G = p.g.G, H = p.g.H, d = p.g.d;
    const int which = (int)(item & 1);
    int64_t rest = item >> 1;
    const int h = (int)(rest % H);
    rest /= H;
    const int j = (int)(rest % p.k);
    const int li = (int)(rest / p.k);

    const int t = p.per_head ? p.idx[((int64_t)li * H + h) * p.k + j] : p.idx[(int64_t)li * p.k + j];
    if (t < 0 || t >= p.n_groups) {
        if (t != -1 && p.flags && lane == 0) atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
        return;
    }
    const int64_t slot = bank_slot(p.g, p.layer_begin + li, t, h);

    const int lpr = d >> 3;          // lanes per token row (8 channels each)
    const int rpi = 32 / lpr;        // rows one warp pass covers
    const int sub = lane / lpr;      // which of those rows this lane serves
    const int cl = lane - sub * lpr; // channel block of this lane

    float s[8], m[8];
    {
        const float4 *sp = reinterpret_cast<const float4 *>((which ? p.scale_v : p.scale_k) + slot * d + cl * 8);
        const float4 *mp = reinterpret_cast<const float4 *>((which ? p.zero_v : p.zero_k) + slot * d + cl * 8);
        const float4 s0 = __ldg(sp), s1 = __ldg(sp + 1), m0 = __ldg(mp), m1 = __ldg(mp + 1);
        s[0] = s0.x; s[1] = s0.y; s[2] = s0.z; s[3] = s0.w; s[4] = s1.x; s[5] = s1.y; s[6] = s1.z; s[7] = s1.w;
        m[0] = m0.x; m[1] = m0.y; m[2] = m0.z; m[3] = m0.w; m[4] = m1.x; m[5] = m1.y; m[6] = m1.z; m[7] = m1.w;
    }
    const uint32_t *codes = reinterpret_cast<const uint32_t *>((which ? p.codes_v : p.codes_k) +
                                                               slot * (int64_t)G * p.g.row_bytes) + cl;
    const int wpr = p.g.row_bytes >> 2;  // 32-bit words per packed row
    OT *out = reinterpret_cast<OT *>(which ? p.va : p.ka) + (int64_t)li * p.sl + (int64_t)h * p.sh +
              ((int64_t)p.token_offset + (int64_t)j * G) * p.st + cl * 8;

    constexpr int kBatch = 8;  // rows whose code words are in flight together, per lane
    for (int r0 = sub; r0 < G; r0 += rpi * kBatch) {
        uint32_t w[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int r = r0 + b * rpi;
            if (r < G) w[b] = __ldg(codes + (int64_t)r * wpr);
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int r = r0 + b * rpi;
            if (r < G) {
                float v[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    // 2^23 + nibble as a float, minus 2^23: exact integer-to-float without a conversion
                    const float code = __uint_as_float(0x4B000000u | ((w[b] >> (4 * c)) & 15u)) - 8388608.0f;
                    v[c] = __fmaf_rn(code, s[c], m[c]);
                }
                uint4 o;
                o.x = pack2<OT>(v[0], v[1]);
                o.y = pack2<OT>(v[2], v[3]);
                o.z = pack2<OT>(v[4], v[5]);
                o.w = pack2<OT>(v[6], v[7]);
                *reinterpret_cast<uint4 *>(out + (int64_t)r * p.st) = o;
            }
        }
    }
}

}  // namespace stom

using namespace stom;

extern "C" int32_t stom_oqm_dequant_gather(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                           int32_t layer_begin, int32_t layer_count,
                                           const int32_t *idx, int32_t k, int32_t n_groups,
                                           void *k_active, void *v_active, int32_t out_dtype,
                                           int64_t stride_layer, int64_t stride_head, int64_t stride_token,
                                           int32_t token_offset, uint32_t *dev_flags, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if ((rc = check_store(store))) return rc;
    if ((rc = check_layers(cfg, layer_begin, layer_count))) return rc;
    if (!idx || !k_active || !v_active || k < 1 || n_groups < 0 || token_offset < 0) return STOM_ERR_INVALID_ARG;
    if (n_groups > cfg->capacity_groups) return STOM_ERR_CAPACITY;
    if (out_dtype != STOM_BF16 && out_dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    if (stride_layer < 0 || stride_head < 0 || stride_token < cfg->head_dim) return STOM_ERR_INVALID_ARG;
    if (!aligned16(k_active) || !aligned16(v_active) || (reinterpret_cast<uintptr_t>(idx) & 3u)) return STOM_ERR_ALIGNMENT;
    if (!stride_ok(stride_layer, out_dtype) || !stride_ok(stride_head, out_dtype) || !stride_ok(stride_token, out_dtype))
        return STOM_ERR_ALIGNMENT;
    if (layer_count == 0) return STOM_OK;

    DequantParams p;
    p.idx = idx;
    p.codes_k = store->codes_k; p.codes_v = store->codes_v;
    p.scale_k = store->scale_k; p.zero_k = store->zero_k; p.scale_v = store->scale_v; p.zero_v = store->zero_v;
    p.ka = k_active; p.va = v_active;
    p.sl = stride_layer; p.sh = stride_head; p.st = stride_token;
    p.g = bank_geom(cfg);
    p.layer_begin = layer_begin; p.k = k; p.n_groups = n_groups; p.token_offset = token_offset;
    p.per_head = cfg->score_mode == STOM_SCORE_PER_HEAD;
    p.flags = dev_flags;
    p.n_items = (int64_t)layer_count * k * cfg->n_kv_heads * 2;
    const int64_t blocks = (p.n_items + kDqWarps - 1) / kDqWarps;
    if (blocks > 0x7fffffffLL) return STOM_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (out_dtype == STOM_BF16)
        dequant_gather_kernel<__nv_bfloat16><<<(unsigned)blocks, kDqWarps * 32, 0, s>>>(p);
    else
        dequant_gather_kernel<__half><<<(unsigned)blocks, kDqWarps * 32, 0, s>>>(p);
    return finish_launch();
}
