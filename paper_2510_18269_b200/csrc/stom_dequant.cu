// A4: dequantize the selected groups into the bounded active cache (paper
// Sec. 3.4: Q_4^{-1} = depack * s + m and KV_active = union of the selected
// groups; appendix "Cache reconstruction for decoding").
//
// One warp owns one unit = half the token rows of (layer, selected slot j, kv
// head, K|V): up to ceil(G/2) rows of d/2 packed bytes in, as many rows of d
// 16-bit values out.  A lane owns 8 adjacent channels: it keeps their 8 (s, m)
// pairs in registers for the whole unit, reads 4 bytes of codes per row and
// writes one 16-byte vector per row, so a warp's store instruction covers 512
// contiguous bytes of the active cache.  Output bytes are 3/4 of the traffic.
// All code words of a unit are requested before the first one is used.
//
// A code nibble becomes a float without a conversion instruction: a byte
// permute drops it into the low mantissa byte of 2^23, and subtracting 2^23
// leaves the integer.  The subtraction and fmaf(code, s, m) run two channels
// at a time (f32x2).  The arithmetic per element is exactly fmaf(code, s, m)
// followed by one rounding to the output type.
#include "stom_internal.cuh"

namespace stom {

constexpr int kDqWarps = 4;

struct DequantParams {
    const int32_t *idx;
    const uint8_t *codes_k, *codes_v;
    const void *scale_k, *zero_k, *scale_v, *zero_v;  // elements of g.meta_dtype
    void *ka, *va;
    int64_t sl, sh, st;  // element strides of the active cache: layer, head, token
    BankGeom g;
    int32_t layer_begin, k, n_groups, token_offset, per_head;
    uint32_t *flags;
    int64_t n_units;
};

__device__ __forceinline__ uint64_t dq_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void dq_unpack(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t dq_fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t dq_sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// LPR: lanes per token row (d / 8); BITS: width of a code.
// grid (ceil(4 H / kDqWarps), k, layer_count): a block serves one (layer, slot) and kDqWarps of its 4 H units
// (kv head x keys|values x first|second half of the rows), so no unit index has to be divided out.
template <typename OT, int LPR, int BITS>
__global__ void __launch_bounds__(kDqWarps * 32) dequant_gather_kernel(const DequantParams p) {
    constexpr int RPP = 32 / LPR;          // rows one warp pass covers
    constexpr int kDqMaxRows = 32 / RPP;   // passes that cover half of the largest group (G <= 64)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.g.G, H = p.g.H, d = p.g.d;
    const int u = blockIdx.x * kDqWarps + warp;
    const int half = u & 1, which = (u >> 1) & 1, h = u >> 2;
    if (h >= H) return;
    const int j = blockIdx.y, li = blockIdx.z;

    grid_dependency_wait();  // idx may come from the kernel just ahead in the stream
    const int t = p.per_head ? p.idx[((int64_t)li * H + h) * p.k + j] : p.idx[(int64_t)li * p.k + j];
    if (t < 0 || t >= p.n_groups) {
        if (t != -1 && p.flags && lane == 0) atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
        return;
    }
    const int64_t slot = bank_slot(p.g, p.layer_begin + li, t, h);
    const int sub = lane / LPR;       // which row of a warp pass this lane serves
    const int cl = lane - sub * LPR;  // channel block of this lane
    const int g_half = (G + 1) >> 1;
    const int r_first = (half ? g_half : 0) + sub, r_end = half ? G : g_half;
    const int n_mine = r_first < r_end ? (r_end - r_first + RPP - 1) / RPP : 0;  // rows this lane serves

    // code words of all this lane's rows first, then the statistics
    const uint8_t *crow = (which ? p.codes_v : p.codes_k) + (slot * G + r_first) * (int64_t)p.g.row_bytes;
    const int cstep = RPP * p.g.row_bytes;
    uint32_t w[kDqMaxRows];
#pragma unroll
    for (int b = 0; b < kDqMaxRows; ++b) w[b] = b < n_mine ? load_codes8<BITS>(crow + b * cstep, cl) : 0u;
    uint64_t s2[4], m2[4];
    {
        float sf[8], mf[8];
        load_scale_zero8(which ? p.scale_v : p.scale_k, which ? p.zero_v : p.zero_k, slot * d + cl * 8, p.g.meta_dtype,
                         sf, mf);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            s2[i] = dq_pack(sf[2 * i], sf[2 * i + 1]);
            m2[i] = dq_pack(mf[2 * i], mf[2 * i + 1]);
        }
    }
    OT *out = reinterpret_cast<OT *>(which ? p.va : p.ka) + (int64_t)li * p.sl + (int64_t)h * p.sh +
              ((int64_t)p.token_offset + (int64_t)j * G + r_first) * p.st + cl * 8;
    const int64_t ostep = RPP * p.st;
    const uint64_t two23 = dq_pack(8388608.0f, 8388608.0f);
#pragma unroll
    for (int b = 0; b < kDqMaxRows; ++b) {
        if (b >= n_mine) break;
        uint32_t f[8], o[4];
        code_floats8<BITS>(w[b], f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint64_t code = dq_sub2(dq_pack(__uint_as_float(f[2 * i]), __uint_as_float(f[2 * i + 1])), two23);
            float v0, v1;
            dq_unpack(dq_fma2(code, s2[i], m2[i]), v0, v1);
            o[i] = pack2<OT>(v0, v1);
        }
        *reinterpret_cast<uint4 *>(out) = make_uint4(o[0], o[1], o[2], o[3]);
        out += ostep;
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
    return dequant_gather_launch(cfg, store, layer_begin, layer_count, idx, k, n_groups, k_active, v_active, out_dtype,
                                 stride_layer, stride_head, stride_token, token_offset, dev_flags, stream, false);
}

int32_t stom::dequant_gather_launch(const stom_oqm_config *cfg, const stom_oqm_store *store, int32_t layer_begin,
                                    int32_t layer_count, const int32_t *idx, int32_t k, int32_t n_groups,
                                    void *k_active, void *v_active, int32_t out_dtype, int64_t stride_layer,
                                    int64_t stride_head, int64_t stride_token, int32_t token_offset,
                                    uint32_t *dev_flags, void *stream, bool after_producer) {
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
    p.n_units = (int64_t)layer_count * k * cfg->n_kv_heads * 4;  // x (keys | values) x (first | second half of the rows)
    if (k > 65535 || layer_count > 65535) return STOM_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const dim3 nb((unsigned)((cfg->n_kv_heads * 4 + kDqWarps - 1) / kDqWarps), (unsigned)k, (unsigned)layer_count);
    const unsigned nt = kDqWarps * 32;
    const bool bf = out_dtype == STOM_BF16;
    cudaError_t le = cudaSuccess;
#define STOM_DQ_KERNEL(OT_, LPR_, BITS_)                                                               \
    do {                                                                                               \
        if (after_producer) le = launch_after_producer(dequant_gather_kernel<OT_, LPR_, BITS_>, nb, dim3(nt), 0, s, p); \
        else dequant_gather_kernel<OT_, LPR_, BITS_><<<nb, nt, 0, s>>>(p);                             \
    } while (0)
#define STOM_DQ_LAUNCH(LPR_)                                                                           \
    do {                                                                                               \
        if (cfg->bits == 4) {                                                                          \
            if (bf) STOM_DQ_KERNEL(__nv_bfloat16, LPR_, 4);                                            \
            else STOM_DQ_KERNEL(__half, LPR_, 4);                                                      \
        } else {                                                                                       \
            if (bf) STOM_DQ_KERNEL(__nv_bfloat16, LPR_, 2);                                            \
            else STOM_DQ_KERNEL(__half, LPR_, 2);                                                      \
        }                                                                                              \
    } while (0)
    switch (cfg->head_dim) {
    case 64: STOM_DQ_LAUNCH(8); break;
    case 128: STOM_DQ_LAUNCH(16); break;
    case 256: STOM_DQ_LAUNCH(32); break;
    default: return STOM_ERR_SHAPE;
    }
#undef STOM_DQ_KERNEL
#undef STOM_DQ_LAUNCH
    if (le != cudaSuccess) {
        set_last_cuda_error(le);
        return STOM_ERR_CUDA;
    }
    return finish_launch();
}
