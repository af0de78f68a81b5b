// A1: group quantizer + representative key (paper Sec. 3.4: Q_4, (s_t, m_t),
// k-bar; appendix "Layer-wise vision memory").
//
// One warp owns one tile = the G tokens x d channels of one (layer, frame,
// kv head) of K or of V.  Lane `lane` owns CPL = d/32 adjacent channels of
// every token row, so the per-channel min / max / sum over the G tokens are
// plain per-lane register reductions: no shared-memory reduction, no block
// barrier, and all G row loads of the tile are in flight at once.  The tile
// stays in registers between the statistics pass and the coding pass, so HBM
// is read exactly once.  Packed codes are staged per warp in shared memory and
// written back with 16-byte stores.
//
// Bit-exactness of the codes: the contract is code = rne(fl((x - m) / s)) in
// binary32 with a true division.  A hardware-exact division per element would
// make the kernel instruction-bound, so the quotient is formed with the
// correctly rounded reciprocal y = rn(1/s) and two residual corrections
//     q0 = rn(diff*y); e = rn(diff - q0*s); q1 = rn(q0 + e*y);
//     e = rn(diff - q1*s); q2 = rn(q1 + e*y)
// (q1 is a faithful quotient, and a faithful quotient corrected once more with
// an exact FMA residual and a correctly rounded reciprocal is the correctly
// rounded quotient -- Markstein's division theorem), followed by the
// add-magic-constant trick for round-half-even.  Channels whose scale is zero
// or outside [2^-60, 2^60] take a slow path with the IEEE division.
#include "stom_internal.cuh"

namespace stom {

constexpr int kQuantWarps = 4;

struct QuantParams {
    const void *K, *V, *Ksum;
    const int32_t *token_idx;
    int64_t sl, sg, sh, st;  // element strides: layer, group(frame), head, token
    uint8_t *codes_k, *codes_v;
    float *scale_k, *zero_k, *scale_v, *zero_v, *rep_key, *rep_norm2;
    BankGeom g;
    int32_t layer_begin, group_begin, F, n_in;
    uint32_t *flags;
    int64_t n_tiles;
};

template <int N>
__device__ __forceinline__ void store_floats(float *dst, const float (&v)[N]) {
    if constexpr (N == 2) {
        *reinterpret_cast<float2 *>(dst) = make_float2(v[0], v[1]);
    } else {
#pragma unroll
        for (int i = 0; i < N / 4; ++i)
            reinterpret_cast<float4 *>(dst)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    }
}

// code of one element on the fast path (scale in the safe range, reciprocal exact-rounded)
__device__ __forceinline__ uint32_t code_fast(float x, float m, float s, float y) {
    const float diff = __fsub_rn(x, m);
    float q = __fmul_rn(diff, y);
    float e = __fmaf_rn(-q, s, diff);
    q = __fmaf_rn(e, y, q);
    e = __fmaf_rn(-q, s, diff);
    q = __fmaf_rn(e, y, q);
    // 1.5 * 2^23: adding it rounds q to an integer (ties to even) in the low mantissa bits
    const float u = __fadd_rn(q, 12582912.0f);
    return __float_as_uint(u) & 15u;
}

// IEEE division; s == 0 marks a constant (or underflowing) channel whose codes are all 0
__device__ __forceinline__ uint32_t code_slow(float x, float m, float s) {
    if (s == 0.0f) return 0u;
    const float t = __fdiv_rn(__fsub_rn(x, m), s);
    float r = rintf(t);
    r = fminf(fmaxf(r, 0.0f), 15.0f);
    return (uint32_t)r;
}

template <typename T, int CPL, int MAXR, bool RESIDENT>
__global__ void __launch_bounds__(kQuantWarps * 32) quantize_kernel(const QuantParams p) {
    constexpr int W = CPL * (int)sizeof(T) / 4;  // 32-bit words one lane loads per row
    extern __shared__ __align__(16) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t tile = (int64_t)blockIdx.x * kQuantWarps + warp;
    if (tile >= p.n_tiles) return;  // whole warp leaves together; no block barrier is used below

    const int G = p.g.G, H = p.g.H, d = p.g.d;
    const int which = (int)(tile & 1);  // 0: keys, 1: values
    int64_t rest = tile >> 1;
    const int h = (int)(rest % H);
    rest /= H;
    const int f = (int)(rest % p.F);
    const int li = (int)(rest / p.F);

    // token row of every group member (identity, or the caller's keep list)
    int tok_lo = lane, tok_hi = lane + 32;
    if (p.token_idx) {
        const int32_t *ti = p.token_idx + (int64_t)f * G;
        bool bad = false;
        if (lane < G) {
            int v = ti[lane];
            bad |= (v < 0 || v >= p.n_in);
            tok_lo = min(max(v, 0), p.n_in - 1);
        }
        if (lane + 32 < G) {
            int v = ti[lane + 32];
            bad |= (v < 0 || v >= p.n_in);
            tok_hi = min(max(v, 0), p.n_in - 1);
        }
        if (bad && p.flags) atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
    }
    const bool has_idx = p.token_idx != nullptr;  // warp-uniform
    auto tok_of = [&](int i) -> int {
        return has_idx ? __shfl_sync(0xffffffffu, i < 32 ? tok_lo : tok_hi, i & 31) : i;
    };

    const int64_t base = (int64_t)li * p.sl + (int64_t)f * p.sg + (int64_t)h * p.sh + lane * CPL;
    const T *src = reinterpret_cast<const T *>(which ? p.V : p.K) + base;

    float mn[CPL], mx[CPL], sum[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        mn[j] = INFINITY;
        mx[j] = -INFINITY;
        sum[j] = 0.0f;
    }

    Words<W> raw[RESIDENT ? MAXR : 1];
    if constexpr (RESIDENT) {
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            const int tok = tok_of(i);
            if (i < G) raw[i] = load_words<W>(src + (int64_t)tok * p.st);
        }
#pragma unroll
        for (int i = 0; i < MAXR; ++i) {
            if (i < G) {
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
                    const float x = elem_of<T, W>(raw[i], j);
                    mn[j] = fminf(mn[j], x);
                    mx[j] = fmaxf(mx[j], x);
                    sum[j] += x;
                }
            }
        }
    } else {
#pragma unroll 8
        for (int i = 0; i < MAXR; ++i) {
            const int tok = tok_of(i);
            if (i < G) {
                const Words<W> r = load_words<W>(src + (int64_t)tok * p.st);
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
                    const float x = elem_of<T, W>(r, j);
                    mn[j] = fminf(mn[j], x);
                    mx[j] = fmaxf(mx[j], x);
                    sum[j] += x;
                }
            }
        }
    }

    // scale, offset, reciprocal
    float s[CPL], y[CPL];
    bool safe = true;
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        s[j] = __fdiv_rn(__fsub_rn(mx[j], mn[j]), 15.0f);
        safe &= (s[j] > 8.673617379884035e-19f) && (s[j] < 1.152921504606847e18f);  // (2^-60, 2^60)
        y[j] = __frcp_rn(s[j]);
    }
    safe = __all_sync(0xffffffffu, safe);

    // coding pass -> per-warp staging buffer
    const int row_bytes = p.g.row_bytes;
    uint8_t *stage = smem + (size_t)warp * G * row_bytes;
    auto emit = [&](int i, uint32_t cw) {
        if constexpr (CPL == 8) *reinterpret_cast<uint32_t *>(stage + i * row_bytes + lane * 4) = cw;
        else if constexpr (CPL == 4) *reinterpret_cast<uint16_t *>(stage + i * row_bytes + lane * 2) = (uint16_t)cw;
        else stage[i * row_bytes + lane] = (uint8_t)cw;
    };
    auto code_row = [&](int i, const Words<W> &r) {
        uint32_t cw = 0;
        if (safe) {
#pragma unroll
            for (int j = 0; j < CPL; ++j) cw |= code_fast(elem_of<T, W>(r, j), mn[j], s[j], y[j]) << (4 * j);
        } else {
#pragma unroll
            for (int j = 0; j < CPL; ++j) cw |= code_slow(elem_of<T, W>(r, j), mn[j], s[j]) << (4 * j);
        }
        emit(i, cw);
    };
    if constexpr (RESIDENT) {
#pragma unroll
        for (int i = 0; i < MAXR; ++i)
            if (i < G) code_row(i, raw[i]);
    } else {
#pragma unroll 4
        for (int i = 0; i < MAXR; ++i) {
            const int tok = tok_of(i);
            if (i < G) code_row(i, load_words<W>(src + (int64_t)tok * p.st));
        }
    }

    const int l = p.layer_begin + li, t = p.group_begin + f;
    const int64_t slot = bank_slot(p.g, l, t, h);

    // statistics
    store_floats<CPL>((which ? p.scale_v : p.scale_k) + slot * d + lane * CPL, s);
    store_floats<CPL>((which ? p.zero_v : p.zero_k) + slot * d + lane * CPL, mn);

    // representative key (keys only): mean over the G tokens, and its squared norm per head
    if (!which) {
        if (p.Ksum) {
            const T *ks = reinterpret_cast<const T *>(p.Ksum) + base;
#pragma unroll
            for (int j = 0; j < CPL; ++j) sum[j] = 0.0f;
#pragma unroll 8
            for (int i = 0; i < MAXR; ++i) {
                const int tok = tok_of(i);
                if (i < G) {
                    const Words<W> r = load_words<W>(ks + (int64_t)tok * p.st);
#pragma unroll
                    for (int j = 0; j < CPL; ++j) sum[j] += elem_of<T, W>(r, j);
                }
            }
        }
        float kb[CPL], n2 = 0.0f;
        const float Gf = (float)G;
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
            kb[j] = __fdiv_rn(sum[j], Gf);
            n2 = fmaf(kb[j], kb[j], n2);
        }
        store_floats<CPL>(p.rep_key + slot * d + lane * CPL, kb);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
        if (lane == 0) p.rep_norm2[slot] = n2;
    }

    // staged codes -> bank, 16 bytes per lane per step
    __syncwarp();
    uint8_t *dst = (which ? p.codes_v : p.codes_k) + slot * (int64_t)G * row_bytes;
    const int n16 = G * row_bytes / 16;
    for (int c = lane; c < n16; c += 32)
        reinterpret_cast<uint4 *>(dst)[c] = reinterpret_cast<const uint4 *>(stage)[c];
}

template <typename T, int CPL, int MAXR, bool RESIDENT>
static int32_t launch_one(const QuantParams &p, cudaStream_t stream) {
    const int64_t blocks = (p.n_tiles + kQuantWarps - 1) / kQuantWarps;
    if (blocks > 0x7fffffffLL) return STOM_ERR_SHAPE;
    const size_t smem = (size_t)kQuantWarps * p.g.G * p.g.row_bytes;
    quantize_kernel<T, CPL, MAXR, RESIDENT><<<(unsigned)blocks, kQuantWarps * 32, smem, stream>>>(p);
    return finish_launch();
}

template <typename T>
static int32_t launch_for_type(const QuantParams &p, cudaStream_t stream) {
    const int G = p.g.G;
    // register budget: keep the tile resident while it costs at most 128 registers per lane
    constexpr bool wide = sizeof(T) == 4;
    switch (p.g.d) {
    case 128:
        if (G <= 16) return launch_one<T, 4, 16, true>(p, stream);
        if (G <= 32) return launch_one<T, 4, 32, true>(p, stream);
        if (G <= 40) return launch_one<T, 4, 40, !wide>(p, stream);
        if (G <= 48) return launch_one<T, 4, 48, !wide>(p, stream);
        if (G <= 56) return launch_one<T, 4, 56, !wide>(p, stream);
        return launch_one<T, 4, 64, !wide>(p, stream);
    case 64:
        return launch_one<T, 2, 64, !wide>(p, stream);
    case 256:
        return launch_one<T, 8, 64, false>(p, stream);
    default:
        return STOM_ERR_SHAPE;
    }
}

}  // namespace stom

using namespace stom;

extern "C" int32_t stom_oqm_quantize_frame(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                           int32_t layer_begin, int32_t layer_count,
                                           int32_t group_begin, int32_t group_count,
                                           const void *K, const void *V,
                                           int64_t stride_layer, int64_t stride_group,
                                           int64_t stride_head, int64_t stride_token,
                                           const void *K_summary, const int32_t *token_idx,
                                           int32_t tokens_per_frame_in, uint32_t *dev_flags, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if ((rc = check_store(store))) return rc;
    if ((rc = check_layers(cfg, layer_begin, layer_count))) return rc;
    if (group_begin < 0 || group_count < 0) return STOM_ERR_INVALID_ARG;
    if ((int64_t)group_begin + group_count > cfg->capacity_groups) return STOM_ERR_CAPACITY;
    if (!K || !V) return STOM_ERR_INVALID_ARG;
    if (token_idx && tokens_per_frame_in < 1) return STOM_ERR_INVALID_ARG;
    if (stride_layer < 0 || stride_group < 0 || stride_head < 0 || stride_token < 0) return STOM_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || (K_summary && !aligned16(K_summary))) return STOM_ERR_ALIGNMENT;
    if (token_idx && (reinterpret_cast<uintptr_t>(token_idx) & 3u)) return STOM_ERR_ALIGNMENT;
    const int dt = cfg->kv_dtype;
    if (!stride_ok(stride_layer, dt) || !stride_ok(stride_group, dt) || !stride_ok(stride_head, dt) ||
        !stride_ok(stride_token, dt))
        return STOM_ERR_ALIGNMENT;
    if (layer_count == 0 || group_count == 0) return STOM_OK;

    QuantParams p;
    p.K = K; p.V = V; p.Ksum = K_summary; p.token_idx = token_idx;
    p.sl = stride_layer; p.sg = stride_group; p.sh = stride_head; p.st = stride_token;
    p.codes_k = store->codes_k; p.codes_v = store->codes_v;
    p.scale_k = store->scale_k; p.zero_k = store->zero_k; p.scale_v = store->scale_v; p.zero_v = store->zero_v;
    p.rep_key = store->rep_key; p.rep_norm2 = store->rep_norm2;
    p.g = bank_geom(cfg);
    p.layer_begin = layer_begin; p.group_begin = group_begin; p.F = group_count; p.n_in = tokens_per_frame_in;
    p.flags = dev_flags;
    p.n_tiles = (int64_t)layer_count * group_count * cfg->n_kv_heads * 2;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (dt) {
    case STOM_BF16: return launch_for_type<__nv_bfloat16>(p, s);
    case STOM_FP16: return launch_for_type<__half>(p, s);
    default: return launch_for_type<float>(p, s);
    }
}
