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

// ---- packed binary32 pairs: sm_100 executes add/sub/mul/fma on two floats per instruction
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Two adjacent channels at once: x - m, the doubly corrected quotient, the rounding add.  Returns the two
// floats 1.5*2^23 + code as a pair; `acc` receives x added to the running sums when SUM is set.
template <bool SUM>
__device__ __forceinline__ uint64_t code_pair(uint64_t x, uint64_t m, uint64_t neg_s, uint64_t y, uint64_t magic,
                                              uint64_t &acc) {
    if constexpr (SUM) acc = add2(acc, x);
    const uint64_t diff = sub2(x, m);
    uint64_t q = mul2(diff, y);
    uint64_t e = fma2(q, neg_s, diff);
    q = fma2(e, y, q);
    e = fma2(q, neg_s, diff);
    q = fma2(e, y, q);
    return add2(q, magic);
}

// LPR: lanes per token row (d / 8); P: rows a thread owns; EXACT: P * rows-per-pass == G (no ragged last pass).
// blockDim.x = 32 * warps.  grid = (2 * H, frames, layers): x = kv head * 2 + (0: keys, 1: values).
template <typename T, int LPR, int P, bool EXACT>
__global__ void __launch_bounds__(kMaxWarps * 32) quantize_kernel(const QuantParams p) {
    constexpr int W = 8 * (int)sizeof(T) / 4;  // 32-bit words of one thread's 8 channels: 4 or 8
    constexpr int RPW = 32 / LPR;              // rows one warp covers per pass
    constexpr int D = LPR * 8;
    __shared__ __align__(16) float part_mn[kMaxWarps][D], part_mx[kMaxWarps][D], part_sum[kMaxWarps][D];
    __shared__ __align__(16) float ch_s[D], ch_y[D], ch_m[D];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
    const int sub = lane / LPR, cl = lane - sub * LPR;
    const int rpp = nwarps * RPW;  // rows per pass of the whole block
    const int rbase = warp * RPW + sub;
    const int G = p.g.G;

    const int which = blockIdx.x & 1, h = blockIdx.x >> 1, f = blockIdx.y, li = blockIdx.z;
    const int64_t base = (int64_t)li * p.sl + (int64_t)f * p.sg + (int64_t)h * p.sh + cl * 8;
    const T *src = reinterpret_cast<const T *>(which ? p.V : p.K) + base;
    const bool want_sum = !which;              // block-uniform: keys carry the representative key
    const bool own_sum = want_sum && !p.Ksum;  // sums come from the tile itself

    // ---- load the thread's rows (all requests issued before any use).  A row past the end of a ragged
    //      last pass re-reads row G-1: harmless for min/max, masked out of sums and stores.
    Words<W> raw[P];
    int64_t row_off[P];
#pragma unroll
    for (int i = 0; i < P; ++i) {
        int r = i * rpp + rbase;
        if constexpr (!EXACT) r = min(r, G - 1);
        int tok = r;
        if (p.token_idx) {
            const int v = p.token_idx[(int64_t)f * G + r];
            if ((v < 0 || v >= p.n_in) && p.flags) atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
            tok = min(max(v, 0), p.n_in - 1);
        }
        row_off[i] = (int64_t)tok * p.st;
        raw[i] = load_words<W>(src + row_off[i]);
    }

    // ---- pass 1: min / max per channel over this thread's rows (two values per word for 16-bit types)
    uint32_t mnw[W], mxw[W];
#pragma unroll
    for (int j = 0; j < W; ++j) mnw[j] = mxw[j] = raw[0].w[j];
#pragma unroll
    for (int i = 1; i < P; ++i) {
#pragma unroll
        for (int j = 0; j < W; ++j) {
            mnw[j] = WordOps<T>::vmin(mnw[j], raw[i].w[j]);
            mxw[j] = WordOps<T>::vmax(mxw[j], raw[i].w[j]);
        }
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {  // rows of the same warp
#pragma unroll
        for (int j = 0; j < W; ++j) {
            mnw[j] = WordOps<T>::vmin(mnw[j], __shfl_xor_sync(0xffffffffu, mnw[j], o));
            mxw[j] = WordOps<T>::vmax(mxw[j], __shfl_xor_sync(0xffffffffu, mxw[j], o));
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
        }
    }
    __syncthreads();

    // ---- owners: thread c finishes the statistics of channel c
    const int64_t slot = bank_slot(p.g, p.layer_begin + li, p.group_begin + f, h);
    bool safe = true;
    for (int c = tid; c < D; c += blockDim.x) {
        float mn = part_mn[0][c], mx = part_mx[0][c];
        for (int w = 1; w < nwarps; ++w) {
            mn = fminf(mn, part_mn[w][c]);
            mx = fmaxf(mx, part_mx[w][c]);
        }
        const float s = __fdiv_rn(__fsub_rn(mx, mn), 15.0f);
        safe &= (s > 8.673617379884035e-19f) && (s < 1.152921504606847e18f);  // (2^-60, 2^60)
        ch_s[c] = s;
        ch_y[c] = __frcp_rn(s);
        ch_m[c] = mn;
        (which ? p.scale_v : p.scale_k)[slot * D + c] = s;
        (which ? p.zero_v : p.zero_k)[slot * D + c] = mn;
    }
    safe = __syncthreads_and(safe);

    // ---- pass 2: codes (and, for keys, the channel sums of the rows as a by-product)
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
    uint64_t sum2[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) sum2[j] = 0ull;  // (+0, +0)

    if (safe) {
        uint64_t m2[4], ns2[4], y2[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            m2[j] = pack_f2(m[2 * j], m[2 * j + 1]);
            ns2[j] = pack_f2(-s[2 * j], -s[2 * j + 1]);
            y2[j] = pack_f2(y[2 * j], y[2 * j + 1]);
        }
        const uint64_t magic = pack_f2(12582912.0f, 12582912.0f);  // 1.5 * 2^23: rounds to integer, ties to even
        // every float 1.5*2^23 + code has the bit pattern 0x4B400000 + code; summing pattern * 16^j over the 8
        // channels and removing the constant part leaves the 8 nibbles in place (they cannot carry into each other)
        constexpr uint32_t kBias = 0x4B400000u * 0x11111111u;
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const int r = i * rpp + rbase;
            const bool valid = EXACT || r < G;
            uint32_t cw = 0u - kBias;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float x0, x1;
                if constexpr (sizeof(T) == 4) {
                    x0 = __uint_as_float(raw[i].w[2 * j]);
                    x1 = __uint_as_float(raw[i].w[2 * j + 1]);
                } else {
                    unpack2<T>(raw[i].w[j], x0, x1);
                }
                uint64_t x = pack_f2(x0, x1);
                uint64_t u;
                if (own_sum) {
                    if (!EXACT && !valid) x = 0ull;  // a padded row adds (+0, +0) to the sums; its codes are dropped
                    u = code_pair<true>(x, m2[j], ns2[j], y2[j], magic, sum2[j]);
                } else {
                    u = code_pair<false>(x, m2[j], ns2[j], y2[j], magic, sum2[j]);
                }
                float u0, u1;
                unpack_f2(u, u0, u1);
                cw += __float_as_uint(u0) << (8 * j);
                cw += __float_as_uint(u1) << (8 * j + 4);
            }
            if (valid) dst[(int64_t)r * LPR] = cw;
        }
    } else {
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const int r = i * rpp + rbase;
            const bool valid = EXACT || r < G;
            uint32_t cw = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float x = elem_of<T, W>(raw[i], j);
                cw |= code_slow(x, m[j], s[j]) << (4 * j);
                if (own_sum && valid) {
                    float a0, a1;
                    unpack_f2(sum2[j >> 1], a0, a1);
                    if (j & 1) a1 += x; else a0 += x;
                    sum2[j >> 1] = pack_f2(a0, a1);
                }
            }
            if (valid) dst[(int64_t)r * LPR] = cw;
        }
    }
    if (!want_sum) return;  // block-uniform

    // ---- representative key: mean over the G tokens of the keys (or of the pre-rotary keys), |k-bar_h|^2
    if (!own_sum) {
        const T *ks = reinterpret_cast<const T *>(p.Ksum) + base;
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const int r = i * rpp + rbase;
            const Words<W> kr = load_words<W>(ks + row_off[i]);
            if (EXACT || r < G) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    sum2[j] = add2(sum2[j], pack_f2(elem_of<T, W>(kr, 2 * j), elem_of<T, W>(kr, 2 * j + 1)));
            }
        }
    }
    float sum[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) unpack_f2(sum2[j], sum[2 * j], sum[2 * j + 1]);
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < 8; ++j) sum[j] += __shfl_xor_sync(0xffffffffu, sum[j], o);
    }
    if (sub == 0) {
#pragma unroll
        for (int j = 0; j < 8; j += 4)
            *reinterpret_cast<float4 *>(&part_sum[warp][cl * 8 + j]) = make_float4(sum[j], sum[j + 1], sum[j + 2], sum[j + 3]);
    }
    __syncthreads();
    if (warp == 0) {  // one warp finishes all D channels, so the norm needs no further block barrier
        float n2 = 0.0f;
        const float Gf = (float)G;
#pragma unroll
        for (int c = lane; c < D; c += 32) {
            float sm = part_sum[0][c];
            for (int w = 1; w < nwarps; ++w) sm += part_sum[w][c];
            const float kb = __fdiv_rn(sm, Gf);
            p.rep_key[slot * D + c] = kb;
            n2 = fmaf(kb, kb, n2);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
        if (lane == 0) p.rep_norm2[slot] = n2;
    }
}

template <typename T, int LPR, int P>
static void launch_exact(const QuantParams &p, dim3 grid, unsigned block, bool exact, cudaStream_t stream) {
    if (exact) quantize_kernel<T, LPR, P, true><<<grid, block, 0, stream>>>(p);
    else quantize_kernel<T, LPR, P, false><<<grid, block, 0, stream>>>(p);
}

template <typename T, int LPR>
static int32_t launch_lpr(const QuantParams &p0, int layer_count, cudaStream_t stream) {
    constexpr int RPW = 32 / LPR;
    // block shape: the (warps, P) pair that covers G rows with the least padding, P <= 8; ties -> more warps
    const int G = p0.g.G;
    int best_w = kMaxWarps, best_p = 8, best_pad = 1 << 30;
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
    const unsigned block = best_w * 32;
    const bool exact = best_pad == 0;
    constexpr int kMaxY = 65535;  // grid.y limit: longer frame ranges are launched in slices
    for (int f0 = 0; f0 < p0.F; f0 += kMaxY) {
        QuantParams p = p0;
        const int nf = p0.F - f0 < kMaxY ? p0.F - f0 : kMaxY;
        const int64_t shift = (int64_t)f0 * p.sg * (int64_t)sizeof(T);
        p.K = static_cast<const uint8_t *>(p.K) + shift;
        p.V = static_cast<const uint8_t *>(p.V) + shift;
        if (p.Ksum) p.Ksum = static_cast<const uint8_t *>(p.Ksum) + shift;
        if (p.token_idx) p.token_idx += (int64_t)f0 * G;
        p.group_begin += f0;
        p.F = nf;
        const dim3 grid(2 * p.g.H, nf, layer_count);
        switch (best_p) {
        case 1: launch_exact<T, LPR, 1>(p, grid, block, exact, stream); break;
        case 2: launch_exact<T, LPR, 2>(p, grid, block, exact, stream); break;
        case 3: launch_exact<T, LPR, 3>(p, grid, block, exact, stream); break;
        case 4: launch_exact<T, LPR, 4>(p, grid, block, exact, stream); break;
        case 5: launch_exact<T, LPR, 5>(p, grid, block, exact, stream); break;
        case 6: launch_exact<T, LPR, 6>(p, grid, block, exact, stream); break;
        case 7: launch_exact<T, LPR, 7>(p, grid, block, exact, stream); break;
        default: launch_exact<T, LPR, 8>(p, grid, block, exact, stream); break;
        }
        const int32_t rc = finish_launch();
        if (rc) return rc;
    }
    return STOM_OK;
}

template <typename T>
static int32_t launch_for_type(const QuantParams &p, int layer_count, cudaStream_t stream) {
    switch (p.g.d) {
    case 64: return launch_lpr<T, 8>(p, layer_count, stream);
    case 128: return launch_lpr<T, 16>(p, layer_count, stream);
    case 256: return launch_lpr<T, 32>(p, layer_count, stream);
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
    if (layer_count > 65535 || 2 * cfg->n_kv_heads > 65535) return STOM_ERR_SHAPE;

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
    case STOM_BF16: return launch_for_type<__nv_bfloat16>(p, layer_count, s);
    case STOM_FP16: return launch_for_type<__half>(p, layer_count, s);
    default: return launch_for_type<float>(p, layer_count, s);
    }
}
