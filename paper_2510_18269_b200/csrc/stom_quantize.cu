// A1: group quantizer + representative key (paper Sec. 3.4: Q_4, (s_t, m_t),
// k-bar; appendix "Layer-wise vision memory").
//
// One thread block owns one tile = the G tokens x d channels of one (layer,
// frame, kv head) of K or of V.  A thread owns 8 adjacent channels (16 bytes of
// a 16-bit row) of P rows; the block size is chosen on the host so that
// P * rows-per-pass covers G with the least padding (G = 50, d = 128: 5 warps,
// 10 rows per pass, P = 5).  The tile is loaded once, stays in registers
// between the statistics pass and the coding pass, and the code that is
// unrolled is only P rows long, so it fits the instruction cache.
//   pass 1  per-thread packed min / max (and binary32 sums for keys), a
//           shuffle across the rows of a warp, per-warp partials to shared memory
//   owners  thread c reduces channel c over the warps, computes s, m, 1/s,
//           the representative key, and writes the statistics (coalesced)
//   pass 2  every thread fetches s, 1/s, m of its 8 channels and emits one
//           32-bit word of codes per row
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
// add-magic-constant trick for round-half-even.  Tiles with a channel whose
// scale is zero or outside (2^-60, 2^60) take a slow path with the IEEE division.
#include "stom_internal.cuh"

namespace stom {

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

constexpr int kMaxWarps = 8;

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

// element-wise min / max on one 32-bit word of a row fragment (two 16-bit values or one float)
template <typename T> struct WordOps;
template <> struct WordOps<__nv_bfloat16> {
    static constexpr uint32_t kPosInf = 0x7F807F80u, kNegInf = 0xFF80FF80u;
    static __device__ __forceinline__ uint32_t vmin(uint32_t a, uint32_t b) {
        __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
        return *reinterpret_cast<uint32_t *>(&r);
    }
    static __device__ __forceinline__ uint32_t vmax(uint32_t a, uint32_t b) {
        __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162 *>(&a), *reinterpret_cast<__nv_bfloat162 *>(&b));
        return *reinterpret_cast<uint32_t *>(&r);
    }
};
template <> struct WordOps<__half> {
    static constexpr uint32_t kPosInf = 0x7C007C00u, kNegInf = 0xFC00FC00u;
    static __device__ __forceinline__ uint32_t vmin(uint32_t a, uint32_t b) {
        __half2 r = __hmin2(*reinterpret_cast<__half2 *>(&a), *reinterpret_cast<__half2 *>(&b));
        return *reinterpret_cast<uint32_t *>(&r);
    }
    static __device__ __forceinline__ uint32_t vmax(uint32_t a, uint32_t b) {
        __half2 r = __hmax2(*reinterpret_cast<__half2 *>(&a), *reinterpret_cast<__half2 *>(&b));
        return *reinterpret_cast<uint32_t *>(&r);
    }
};
template <> struct WordOps<float> {
    static constexpr uint32_t kPosInf = 0x7F800000u, kNegInf = 0xFF800000u;
    static __device__ __forceinline__ uint32_t vmin(uint32_t a, uint32_t b) {
        return __float_as_uint(fminf(__uint_as_float(a), __uint_as_float(b)));
    }
    static __device__ __forceinline__ uint32_t vmax(uint32_t a, uint32_t b) {
        return __float_as_uint(fmaxf(__uint_as_float(a), __uint_as_float(b)));
    }
};

// LPR: lanes per token row (d / 8); P: rows a thread owns.  blockDim.x = 32 * warps.
template <typename T, int LPR, int P>
__global__ void __launch_bounds__(kMaxWarps * 32) quantize_kernel(const QuantParams p) {
    constexpr int W = 8 * (int)sizeof(T) / 4;  // 32-bit words of one thread's 8 channels: 4 or 8
    constexpr int RPW = 32 / LPR;              // rows one warp covers per pass
    constexpr int D = LPR * 8;
    __shared__ __align__(16) float part_mn[kMaxWarps][D], part_mx[kMaxWarps][D], part_sum[kMaxWarps][D];
    __shared__ __align__(16) float ch_s[D], ch_y[D], ch_m[D];
    __shared__ float warp_n2[kMaxWarps];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
    const int sub = lane / LPR, cl = lane - sub * LPR;
    const int rpp = nwarps * RPW;  // rows per pass of the whole block
    const int G = p.g.G, H = p.g.H;

    const int64_t tile = blockIdx.x;
    const int which = (int)(tile & 1);  // 0: keys, 1: values
    int64_t rest = tile >> 1;
    const int h = (int)(rest % H);
    rest /= H;
    const int f = (int)(rest % p.F);
    const int li = (int)(rest / p.F);
    const int64_t base = (int64_t)li * p.sl + (int64_t)f * p.sg + (int64_t)h * p.sh + cl * 8;
    const T *src = reinterpret_cast<const T *>(which ? p.V : p.K) + base;
    const bool want_sum = !which;                 // block-uniform
    const bool own_sum = want_sum && !p.Ksum;     // sums come from the tile itself

    // ---- load the thread's rows (all requests issued before any use)
    Words<W> raw[P];
    int64_t row_off[P];
#pragma unroll
    for (int i = 0; i < P; ++i) {
        const int r = i * rpp + warp * RPW + sub;
        int tok = r;
        if (p.token_idx && r < G) {
            const int v = p.token_idx[(int64_t)f * G + r];
            if (v < 0 || v >= p.n_in) {
                if (p.flags) atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
            }
            tok = min(max(v, 0), p.n_in - 1);
        }
        row_off[i] = (int64_t)tok * p.st;
        if (r < G) raw[i] = load_words<W>(src + row_off[i]);
    }

    // ---- pass 1: min / max per channel over this thread's rows (packed for 16-bit types), sums for keys
    uint32_t mnw[W], mxw[W];
    float sum[8];
#pragma unroll
    for (int j = 0; j < W; ++j) {
        mnw[j] = WordOps<T>::kPosInf;
        mxw[j] = WordOps<T>::kNegInf;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) sum[j] = 0.0f;
#pragma unroll
    for (int i = 0; i < P; ++i) {
        const int r = i * rpp + warp * RPW + sub;
        if (r < G) {
#pragma unroll
            for (int j = 0; j < W; ++j) {
                mnw[j] = WordOps<T>::vmin(mnw[j], raw[i].w[j]);
                mxw[j] = WordOps<T>::vmax(mxw[j], raw[i].w[j]);
            }
            if (own_sum) {
#pragma unroll
                for (int j = 0; j < 8; ++j) sum[j] += elem_of<T, W>(raw[i], j);
            }
        }
    }
    if (want_sum && !own_sum) {  // keys averaged from the separate pre-rotary tensor
        const T *ks = reinterpret_cast<const T *>(p.Ksum) + base;
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const int r = i * rpp + warp * RPW + sub;
            if (r < G) {
                const Words<W> kr = load_words<W>(ks + row_off[i]);
#pragma unroll
                for (int j = 0; j < 8; ++j) sum[j] += elem_of<T, W>(kr, j);
            }
        }
    }
    // rows of the same warp
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < W; ++j) {
            mnw[j] = WordOps<T>::vmin(mnw[j], __shfl_xor_sync(0xffffffffu, mnw[j], o));
            mxw[j] = WordOps<T>::vmax(mxw[j], __shfl_xor_sync(0xffffffffu, mxw[j], o));
        }
        if (want_sum) {
#pragma unroll
            for (int j = 0; j < 8; ++j) sum[j] += __shfl_xor_sync(0xffffffffu, sum[j], o);
        }
    }
    if (sub == 0) {
        Words<W> a, b;
#pragma unroll
        for (int j = 0; j < W; ++j) {
            a.w[j] = mnw[j];
            b.w[j] = mxw[j];
        }
#pragma unroll
        for (int j = 0; j < 8; j += 4) {
            *reinterpret_cast<float4 *>(&part_mn[warp][cl * 8 + j]) =
                make_float4(elem_of<T, W>(a, j), elem_of<T, W>(a, j + 1), elem_of<T, W>(a, j + 2), elem_of<T, W>(a, j + 3));
            *reinterpret_cast<float4 *>(&part_mx[warp][cl * 8 + j]) =
                make_float4(elem_of<T, W>(b, j), elem_of<T, W>(b, j + 1), elem_of<T, W>(b, j + 2), elem_of<T, W>(b, j + 3));
            if (want_sum)
                *reinterpret_cast<float4 *>(&part_sum[warp][cl * 8 + j]) = make_float4(sum[j], sum[j + 1], sum[j + 2], sum[j + 3]);
        }
    }
    __syncthreads();

    // ---- owners: thread c finishes channel c
    const int l = p.layer_begin + li, t = p.group_begin + f;
    const int64_t slot = bank_slot(p.g, l, t, h);
    bool safe = true;
    float n2 = 0.0f;
    for (int c = tid; c < D; c += blockDim.x) {
        float mn = part_mn[0][c], mx = part_mx[0][c], sm = want_sum ? part_sum[0][c] : 0.0f;
        for (int w = 1; w < nwarps; ++w) {
            mn = fminf(mn, part_mn[w][c]);
            mx = fmaxf(mx, part_mx[w][c]);
            if (want_sum) sm += part_sum[w][c];
        }
        const float s = __fdiv_rn(__fsub_rn(mx, mn), 15.0f);
        safe &= (s > 8.673617379884035e-19f) && (s < 1.152921504606847e18f);  // (2^-60, 2^60)
        ch_s[c] = s;
        ch_y[c] = __frcp_rn(s);
        ch_m[c] = mn;
        (which ? p.scale_v : p.scale_k)[slot * D + c] = s;
        (which ? p.zero_v : p.zero_k)[slot * D + c] = mn;
        if (want_sum) {
            const float kb = __fdiv_rn(sm, (float)G);
            p.rep_key[slot * D + c] = kb;
            n2 = fmaf(kb, kb, n2);
        }
    }
    if (want_sum) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
        if (lane == 0) warp_n2[warp] = n2;
    }
    safe = __syncthreads_and(safe);
    if (want_sum && tid == 0) {
        float tot = 0.0f;
        for (int w = 0; w < nwarps; ++w) tot += warp_n2[w];
        p.rep_norm2[slot] = tot;
    }

    // ---- pass 2: codes
    float s[8], y[8], m[8];
#pragma unroll
    for (int j = 0; j < 8; j += 4) {
        const float4 a = *reinterpret_cast<const float4 *>(&ch_s[cl * 8 + j]);
        const float4 b = *reinterpret_cast<const float4 *>(&ch_y[cl * 8 + j]);
        const float4 c = *reinterpret_cast<const float4 *>(&ch_m[cl * 8 + j]);
        s[j] = a.x; s[j + 1] = a.y; s[j + 2] = a.z; s[j + 3] = a.w;
        y[j] = b.x; y[j + 1] = b.y; y[j + 2] = b.z; y[j + 3] = b.w;
        m[j] = c.x; m[j + 1] = c.y; m[j + 2] = c.z; m[j + 3] = c.w;
    }
    uint32_t *dst = reinterpret_cast<uint32_t *>((which ? p.codes_v : p.codes_k) + slot * (int64_t)G * p.g.row_bytes) + cl;
#pragma unroll
    for (int i = 0; i < P; ++i) {
        const int r = i * rpp + warp * RPW + sub;
        if (r < G) {
            uint32_t cw = 0;
            if (safe) {
#pragma unroll
                for (int j = 0; j < 8; ++j) cw |= code_fast(elem_of<T, W>(raw[i], j), m[j], s[j], y[j]) << (4 * j);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) cw |= code_slow(elem_of<T, W>(raw[i], j), m[j], s[j]) << (4 * j);
            }
            dst[(int64_t)r * LPR] = cw;
        }
    }
}

template <typename T, int LPR>
static int32_t launch_lpr(const QuantParams &p, cudaStream_t stream) {
    if (p.n_tiles > 0x7fffffffLL) return STOM_ERR_SHAPE;
    constexpr int RPW = 32 / LPR;
    // block shape: the (warps, P) pair that covers G rows with the least padding, P <= 8; ties -> more warps
    const int G = p.g.G;
    int best_w = kMaxWarps, best_p = (G + kMaxWarps * RPW - 1) / (kMaxWarps * RPW), best_pad = 1 << 30;
    for (int w = kMaxWarps; w >= 2; --w) {
        const int P = (G + w * RPW - 1) / (w * RPW);
        if (P > 8) continue;
        const int pad = P * w * RPW - G;
        if (pad < best_pad) {
            best_pad = pad;
            best_w = w;
            best_p = P;
        }
    }
    const unsigned grid = (unsigned)p.n_tiles, block = best_w * 32;
    switch (best_p) {
    case 1: quantize_kernel<T, LPR, 1><<<grid, block, 0, stream>>>(p); break;
    case 2: quantize_kernel<T, LPR, 2><<<grid, block, 0, stream>>>(p); break;
    case 3: quantize_kernel<T, LPR, 3><<<grid, block, 0, stream>>>(p); break;
    case 4: quantize_kernel<T, LPR, 4><<<grid, block, 0, stream>>>(p); break;
    case 5: quantize_kernel<T, LPR, 5><<<grid, block, 0, stream>>>(p); break;
    case 6: quantize_kernel<T, LPR, 6><<<grid, block, 0, stream>>>(p); break;
    case 7: quantize_kernel<T, LPR, 7><<<grid, block, 0, stream>>>(p); break;
    default: quantize_kernel<T, LPR, 8><<<grid, block, 0, stream>>>(p); break;
    }
    return finish_launch();
}

template <typename T>
static int32_t launch_for_type(const QuantParams &p, cudaStream_t stream) {
    switch (p.g.d) {
    case 64: return launch_lpr<T, 8>(p, stream);
    case 128: return launch_lpr<T, 16>(p, stream);
    case 256: return launch_lpr<T, 32>(p, stream);
    default: return STOM_ERR_SHAPE;
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
