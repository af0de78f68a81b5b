/*
 * CPU oracle for StreamingTOM's Online Quantized Memory (OQM).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow restatement of the
 * method, step by step, in the paper's order and notation.  It shares no
 * code, header, table or helper with the CUDA library, and the CUDA library
 * never calls it.  Only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg load it.
 *
 * Every pointer is a HOST pointer.  Floating point that decides an integer
 * (the 4-bit codes) is done in IEEE binary32 exactly as written here; all
 * other reductions (means, norms, dot products, softmax) are done in
 * binary64.  Build with  gcc -O2 -ffp-contract=off -fno-fast-math  so the
 * compiler neither fuses nor reorders the binary32 operations.
 *
 * Passages followed (paper section / equation):
 *   - group quantizer, scale and offset ........ Sec. 3.4 "Online Quantized
 *     Memory", the Q_4 equation and the (s_t, m_t) equation
 *   - representative key ...................... Sec. 3.4 (mean of the keys
 *     before quantization); appendix "Layer-wise vision memory"
 *   - dequantization .......................... Sec. 3.4, the Q_4^{-1} equation
 *   - question embedding, cosine top-K ........ appendix "Question-guided
 *     single-pass retrieval" (the q^(l) equation and the K = min(..) equation)
 *   - active cache ............................ Sec. 3.4, the KV_active
 *     equation; appendix "Cache reconstruction for decoding"
 *   - CTR: temporal similarity, static/dynamic split, budget split, dynamic
 *     selection ............................... Sec. 3.3, the s_t^(i) equation,
 *     the (S_t, D_t) equation, the (k_s, k_d) equation and the TopK half of
 *     the (G_d, G_s) equation.  The Merge half (density-based clustering of
 *     the static tokens) is not restated: the paper gives no definition of it
 *   - storage accounting ...................... Sec. 3.1 memory-growth
 *     equation and its footnote; Sec. 3.2 ratio 4N/G; ablation table "Ratio"
 *
 * Readings taken where the paper is silent (kept in one place so they can be
 * checked by eye):
 *   - forward map: code = clamp(rne((x - m) / s), 0, 15), true division,
 *     round-half-to-even; if s == 0 the channel is constant (or its range
 *     underflows) and every code is 0;
 *   - packing: along the channel axis, even channel in the low nibble;
 *   - inverse map: fmaf(code, s, m), then one rounding to the output type;
 *   - GQA: query head h_q belongs to kv head h_q / (H_q / H_k);
 *   - zero norms: each norm is clamped below by 1e-12 (score becomes 0);
 *   - ties in top-K: the lower group index wins;
 *   - CTR: the first frame of a stream has no predecessor, so none of its
 *     tokens is static (similarity -inf); a zero feature vector has
 *     similarity 0 (norms clamped below by 1e-12, as for the scores); ties in
 *     the saliency TopK go to the lower token index and the selection is
 *     returned in ascending token order;
 *   - 16-bit metadata (meta_dtype = fp16 or bf16; Sec. 4.1 runs the model in
 *     FP16, the (s_t, m_t) equation fixes no storage type): the offset is the
 *     largest 16-bit value <= the channel minimum, the scale the smallest
 *     16-bit value >= fl32((max - m) / levels), and the codes are taken
 *     against THOSE two numbers, so that every code stays in range and the
 *     reconstruction error stays <= s/2 for the stored s; the representative
 *     key is rounded to nearest-even and its norm is the norm of the rounded
 *     vector.  The bank arrays here stay binary32 and hold values that are
 *     exactly representable in the 16-bit type.
 *
 * Pin status: every exported function is pinned by tests that do not call it
 * to produce their own expectation (closed forms, invariants, brute force,
 * library routines, values printed in the paper), except the byte layout of
 * the packed codes (nibble order), which the paper does not fix:
 * "parity unpinned" for the nibble order only.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_ERR_ARG (-1)

enum { ORC_BF16 = 0, ORC_FP16 = 1, ORC_FP32 = 2 };
enum { ORC_PER_LAYER = 0, ORC_PER_HEAD = 1 };

/* Same field order as the CUDA library's config so one Python-side recipe
 * can fill either; declared here independently on purpose. */
typedef struct {
    int32_t n_layers;        /* L   */
    int32_t n_q_heads;       /* H_q */
    int32_t n_kv_heads;      /* H_k */
    int32_t head_dim;        /* d   */
    int32_t group_tokens;    /* G   */
    int32_t capacity_groups; /* groups the store can hold per layer */
    int32_t bits;            /* 4 or 2 */
    int32_t kv_dtype;        /* ORC_BF16 | ORC_FP16 | ORC_FP32 */
    int32_t score_mode;      /* ORC_PER_LAYER | ORC_PER_HEAD */
    int32_t meta_dtype;      /* type s, m and k-bar are stored in: ORC_FP32 (default reading) | ORC_FP16 | ORC_BF16 */
} orc_config;

/* Arrays of the memory bank, all indexed [layer][group][kv head]... */
typedef struct {
    uint8_t *codes_k;  /* [L][cap][H_k][G][d*bits/8] */
    uint8_t *codes_v;  /* same                         */
    float *scale_k;    /* [L][cap][H_k][d]             */
    float *zero_k;     /* [L][cap][H_k][d]             */
    float *scale_v;    /* [L][cap][H_k][d]             */
    float *zero_v;     /* [L][cap][H_k][d]             */
    float *rep_key;    /* [L][cap][H_k][d]  k-bar      */
    float *rep_norm2;  /* [L][cap][H_k]     |k-bar_h|^2 */
} orc_store;

/* ------------------------------------------------------------------ */
/* number formats                                                      */
/* ------------------------------------------------------------------ */

static float bits_to_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static uint32_t f32_to_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

/* bfloat16 is the upper half of a binary32 */
float orc_bf16_to_f32(uint16_t h) { return bits_to_f32((uint32_t)h << 16); }

/* binary32 -> bfloat16, round to nearest, ties to even */
uint16_t orc_f32_to_bf16(float f) {
    uint32_t u = f32_to_bits(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN */
    uint32_t lower = u & 0xffffu;
    uint32_t upper = u >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;
    return (uint16_t)upper;
}

/* IEEE binary16 -> binary32 (exact) */
float orc_f16_to_f32(uint16_t h) {
    uint32_t sign = (uint32_t)(h >> 15) << 31;
    int32_t e = (h >> 10) & 0x1f;
    uint32_t frac = h & 0x3ffu;
    if (e == 0x1f) return bits_to_f32(sign | 0x7f800000u | (frac << 13));
    if (e == 0) {
        /* subnormal: frac * 2^-24 */
        float v = (float)frac * 5.9604644775390625e-08f;
        return sign ? -v : v;
    }
    return bits_to_f32(sign | ((uint32_t)(e - 15 + 127) << 23) | (frac << 13));
}

/* binary32 -> IEEE binary16, round to nearest, ties to even */
uint16_t orc_f32_to_f16(float f) {
    uint32_t u = f32_to_bits(f);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t a = u & 0x7fffffffu;
    if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);  /* NaN */
    if (a >= 0x477ff000u) return (uint16_t)(sign | 0x7c00u); /* >= 65520 rounds to inf */
    double mag = fabs((double)f);
    if (mag < 6.103515625e-05) {
        /* subnormal target: multiples of 2^-24 */
        double q = mag * 16777216.0;
        double r = nearbyint(q); /* ties to even in the default mode */
        return (uint16_t)(sign | (uint16_t)r); /* r == 1024 gives the smallest normal */
    }
    int e;
    double fr = frexp(mag, &e); /* mag = fr * 2^e, fr in [0.5,1) */
    double sig = fr * 2048.0;   /* in [1024, 2048) */
    double r = nearbyint(sig);
    int ee = e - 1;             /* unbiased exponent of the leading bit */
    if (r == 2048.0) { r = 1024.0; ee += 1; }
    return (uint16_t)(sign | (uint16_t)((ee + 15) << 10) | ((uint16_t)r - 1024u));
}

static float load_elem(const void *p, int64_t i, int dtype) {
    switch (dtype) {
    case ORC_BF16: return orc_bf16_to_f32(((const uint16_t *)p)[i]);
    case ORC_FP16: return orc_f16_to_f32(((const uint16_t *)p)[i]);
    default: return ((const float *)p)[i];
    }
}

void orc_convert_to_f32(const void *src, int dtype, int64_t n, float *dst) {
    for (int64_t i = 0; i < n; ++i) dst[i] = load_elem(src, i, dtype);
}

void orc_convert_from_f32(const float *src, int dtype, int64_t n, void *dst) {
    for (int64_t i = 0; i < n; ++i) {
        if (dtype == ORC_BF16) ((uint16_t *)dst)[i] = orc_f32_to_bf16(src[i]);
        else if (dtype == ORC_FP16) ((uint16_t *)dst)[i] = orc_f32_to_f16(src[i]);
        else ((float *)dst)[i] = src[i];
    }
}

/* Nearest-even rounding of a binary32 to the type `dtype`, returned as binary32. */
float orc_round_nearest(float x, int dtype) {
    if (dtype == ORC_BF16) return orc_bf16_to_f32(orc_f32_to_bf16(x));
    if (dtype == ORC_FP16) return orc_f16_to_f32(orc_f32_to_f16(x));
    return x;
}

/* The neighbour of the 16-bit pattern h one step towards -inf (dir < 0) or
 * +inf (dir > 0) on the number line.  Both formats are sign-magnitude, so a
 * step away from zero adds one to the pattern and a step towards zero takes
 * one off; stepping down from +0 lands on the smallest negative subnormal. */
static uint16_t step16(uint16_t h, int dir) {
    int negative = (h & 0x8000u) != 0;
    if ((h & 0x7fffu) == 0) return dir > 0 ? (uint16_t)0x0001u : (uint16_t)0x8001u;
    if ((dir > 0) == !negative) return (uint16_t)(h + 1u); /* away from zero */
    return (uint16_t)(h - 1u);                               /* towards zero   */
}

static float f32_of16(uint16_t h, int dtype) { return dtype == ORC_BF16 ? orc_bf16_to_f32(h) : orc_f16_to_f32(h); }
static uint16_t to16(float x, int dtype) { return dtype == ORC_BF16 ? orc_f32_to_bf16(x) : orc_f32_to_f16(x); }

/* Largest value of the type that is <= x (x finite and inside the type's range). */
float orc_round_down(float x, int dtype) {
    if (dtype == ORC_FP32) return x;
    uint16_t h = to16(x, dtype);
    if (f32_of16(h, dtype) > x) h = step16(h, -1);
    return f32_of16(h, dtype);
}

/* Smallest value of the type that is >= x. */
float orc_round_up(float x, int dtype) {
    if (dtype == ORC_FP32) return x;
    uint16_t h = to16(x, dtype);
    if (f32_of16(h, dtype) < x) h = step16(h, +1);
    return f32_of16(h, dtype);
}

/* ------------------------------------------------------------------ */
/* O1  group quantizer (Sec. 3.4, Q_4 and the (s_t, m_t) equation)     */
/* ------------------------------------------------------------------ */

static int levels_of(int bits) { return (1 << bits) - 1; } /* 15 for 4-bit, 3 for 2-bit */

/*
 * X is one group tensor [H][G][d] in binary32.  Statistics are taken per
 * head and per channel across the G tokens.  codes is [H][G][d] with one
 * code per byte (not yet packed); s and m are [H][d].
 */
void orc_quantize_group(const float *X, int H, int G, int d, int bits, int meta_dtype,
                        uint8_t *codes, float *s, float *m) {
    const float nlev = (float)levels_of(bits);
    for (int h = 0; h < H; ++h) {
        for (int c = 0; c < d; ++c) {
            float mn = X[((int64_t)h * G + 0) * d + c];
            float mx = mn;
            for (int g = 1; g < G; ++g) {
                float x = X[((int64_t)h * G + g) * d + c];
                if (x < mn) mn = x;
                if (x > mx) mx = x;
            }
            mn = orc_round_down(mn, meta_dtype); /* the stored offset; unchanged for binary32 metadata */
            float range = mx - mn;
            float sc = orc_round_up(range / nlev, meta_dtype);
            s[h * d + c] = sc;
            m[h * d + c] = mn;
            for (int g = 0; g < G; ++g) {
                float x = X[((int64_t)h * G + g) * d + c];
                int code = 0;
                if (sc != 0.0f) {
                    float diff = x - mn;
                    float t = diff / sc;
                    float r = nearbyintf(t); /* default mode: ties to even */
                    if (r < 0.0f) r = 0.0f;
                    if (r > nlev) r = nlev;
                    code = (int)r;
                }
                codes[((int64_t)h * G + g) * d + c] = (uint8_t)code;
            }
        }
    }
}

/* Pack one row of d codes: bits=4 -> 2 per byte, bits=2 -> 4 per byte; the
 * lowest channel sits in the lowest bits. */
void orc_pack_row(const uint8_t *codes, int d, int bits, uint8_t *out) {
    int per = 8 / bits;
    for (int j = 0; j < d / per; ++j) {
        unsigned b = 0;
        for (int i = 0; i < per; ++i) b |= (unsigned)codes[j * per + i] << (bits * i);
        out[j] = (uint8_t)b;
    }
}

void orc_unpack_row(const uint8_t *packed, int d, int bits, uint8_t *codes) {
    int per = 8 / bits;
    unsigned mask = (1u << bits) - 1u;
    for (int j = 0; j < d / per; ++j)
        for (int i = 0; i < per; ++i) codes[j * per + i] = (uint8_t)((packed[j] >> (bits * i)) & mask);
}

/* Sec. 3.4, Q_4^{-1}: depack(X) * s + m, evaluated as one fused multiply-add */
float orc_dequant_value(int code, float s, float m) { return fmaf((float)code, s, m); }

/* ------------------------------------------------------------------ */
/* O2  representative key (Sec. 3.4; appendix "Layer-wise vision        */
/*     memory": k_t = (1/G) sum_{i in G_t} K_i)                         */
/* ------------------------------------------------------------------ */

void orc_rep_key(const float *K, int H, int G, int d, int meta_dtype, float *rep, float *norm2) {
    for (int h = 0; h < H; ++h) {
        double n2 = 0.0;
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int g = 0; g < G; ++g) acc += (double)K[((int64_t)h * G + g) * d + c];
            float kb = orc_round_nearest((float)(acc / (double)G), meta_dtype);
            rep[h * d + c] = kb;
            n2 += (double)kb * (double)kb;
        }
        norm2[h] = (float)n2;
    }
}

/* ------------------------------------------------------------------ */
/* store addressing                                                     */
/* ------------------------------------------------------------------ */

static int64_t code_row_bytes(const orc_config *c) { return (int64_t)c->head_dim * c->bits / 8; }
static int64_t codes_off(const orc_config *c, int l, int t, int h) {
    return ((((int64_t)l * c->capacity_groups + t) * c->n_kv_heads + h) * c->group_tokens) * code_row_bytes(c);
}
static int64_t meta_off(const orc_config *c, int l, int t, int h) {
    return (((int64_t)l * c->capacity_groups + t) * c->n_kv_heads + h) * c->head_dim;
}
static int64_t norm_off(const orc_config *c, int l, int t, int h) {
    return ((int64_t)l * c->capacity_groups + t) * c->n_kv_heads + h;
}

static int check_cfg(const orc_config *c) {
    if (!c) return 0;
    if (c->n_layers < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return 0;
    if (c->n_q_heads % c->n_kv_heads) return 0;
    if (c->head_dim < 1 || c->group_tokens < 1 || c->capacity_groups < 1) return 0;
    if (c->bits != 4 && c->bits != 2) return 0;
    if ((c->head_dim * c->bits) % 8) return 0;
    if (c->kv_dtype < 0 || c->kv_dtype > 2) return 0;
    if (c->score_mode < 0 || c->score_mode > 1) return 0;
    if (c->meta_dtype < 0 || c->meta_dtype > 2) return 0;
    return 1;
}

/* ------------------------------------------------------------------ */
/* A1  quantize the groups of newly arrived frames and append them      */
/* ------------------------------------------------------------------ */

/*
 * K, V: element (l, f, h, tok, c) lives at
 *   (l - layer_begin)*stride_layer + f*stride_group + h*stride_head
 *   + tok*stride_token + c            (strides in elements)
 * with tok = token_idx ? token_idx[f*G + g] : g  for g in [0, G).
 * K_summary (nullable) has the same addressing and supplies the keys the
 * representative key is averaged from (keys before rotary embedding).
 * Writes store slots [group_begin, group_begin + group_count) of layers
 * [layer_begin, layer_begin + layer_count); never reads older groups.
 */
int32_t orc_quantize_frame(const orc_config *cfg, const orc_store *st,
                           int32_t layer_begin, int32_t layer_count,
                           int32_t group_begin, int32_t group_count,
                           const void *K, const void *V,
                           int64_t stride_layer, int64_t stride_group,
                           int64_t stride_head, int64_t stride_token,
                           const void *K_summary, const int32_t *token_idx,
                           int32_t tokens_per_frame_in, int32_t n_threads) {
    if (!check_cfg(cfg) || !st || !K || !V) return ORC_ERR_ARG;
    if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > cfg->n_layers) return ORC_ERR_ARG;
    if (group_begin < 0 || group_count < 0 || group_begin + group_count > cfg->capacity_groups) return ORC_ERR_ARG;
    const int H = cfg->n_kv_heads, G = cfg->group_tokens, d = cfg->head_dim;
    if (token_idx) { /* tokens_per_frame_in only bounds token_idx */
        for (int64_t i = 0; i < (int64_t)group_count * G; ++i)
            if (token_idx[i] < 0 || token_idx[i] >= tokens_per_frame_in) return ORC_ERR_ARG;
    }
    const int64_t units = (int64_t)layer_count * group_count;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
    int failed = 0;
#pragma omp parallel for schedule(static)
    for (int64_t u = 0; u < units; ++u) {
        const int li = (int)(u / group_count), f = (int)(u % group_count);
        const int l = layer_begin + li, t = group_begin + f;
        float *X = (float *)malloc(sizeof(float) * (size_t)H * G * d);
        float *Ks = (float *)malloc(sizeof(float) * (size_t)H * G * d);
        uint8_t *codes = (uint8_t *)malloc((size_t)H * G * d);
        if (!X || !Ks || !codes) { failed = 1; free(X); free(Ks); free(codes); continue; }
        for (int which = 0; which < 2; ++which) { /* 0: keys, 1: values */
            const void *src = which ? V : K;
            for (int h = 0; h < H; ++h)
                for (int g = 0; g < G; ++g) {
                    int tok = token_idx ? token_idx[(int64_t)f * G + g] : g;
                    int64_t base = (int64_t)li * stride_layer + (int64_t)f * stride_group +
                                   (int64_t)h * stride_head + (int64_t)tok * stride_token;
                    for (int c = 0; c < d; ++c) {
                        X[((int64_t)h * G + g) * d + c] = load_elem(src, base + c, cfg->kv_dtype);
                        if (!which)
                            Ks[((int64_t)h * G + g) * d + c] =
                                load_elem(K_summary ? K_summary : K, base + c, cfg->kv_dtype);
                    }
                }
            float *s = (which ? st->scale_v : st->scale_k) + meta_off(cfg, l, t, 0);
            float *m = (which ? st->zero_v : st->zero_k) + meta_off(cfg, l, t, 0);
            orc_quantize_group(X, H, G, d, cfg->bits, cfg->meta_dtype, codes, s, m);
            uint8_t *dst = (which ? st->codes_v : st->codes_k) + codes_off(cfg, l, t, 0);
            for (int64_t r = 0; r < (int64_t)H * G; ++r)
                orc_pack_row(codes + r * d, d, cfg->bits, dst + r * code_row_bytes(cfg));
            if (!which)
                orc_rep_key(Ks, H, G, d, cfg->meta_dtype, st->rep_key + meta_off(cfg, l, t, 0),
                            st->rep_norm2 + norm_off(cfg, l, t, 0));
        }
        free(X); free(Ks); free(codes);
    }
    return failed ? ORC_ERR_ARG : ORC_OK;
}

/* ------------------------------------------------------------------ */
/* A2  question embedding and cosine scores (appendix "Question-guided  */
/*     single-pass retrieval")                                          */
/* ------------------------------------------------------------------ */

/*
 * Q element (l, h_q, j, c) at (l-layer_begin)*q_stride_layer + h_q*q_stride_head
 * + j*q_stride_token + c.  qemb is [H_k][d] binary64: the mean over the query
 * heads of each GQA block and over the T_q tokens.
 */
void orc_query_embedding(const orc_config *cfg, const void *Q, int q_dtype, int64_t layer_off,
                         int32_t T_q, int64_t q_stride_head, int64_t q_stride_token, double *qemb) {
    const int H = cfg->n_kv_heads, d = cfg->head_dim, rep = cfg->n_q_heads / cfg->n_kv_heads;
    for (int h = 0; h < H; ++h)
        for (int c = 0; c < d; ++c) {
            double head_acc = 0.0;
            for (int r = 0; r < rep; ++r) {
                int hq = h * rep + r;
                double tok_acc = 0.0;
                for (int j = 0; j < T_q; ++j)
                    tok_acc += (double)load_elem(Q, layer_off + hq * q_stride_head + j * q_stride_token + c, q_dtype);
                head_acc += tok_acc / (double)T_q;
            }
            qemb[h * d + c] = head_acc / (double)rep;
        }
}

/*
 * scores: PER_LAYER -> [layer_count][n_groups]; PER_HEAD -> [layer_count][H_k][n_groups].
 * score = <q, k-bar_t> / (max(|q|, eps) * max(|k-bar_t|, eps)), eps = 1e-12.
 */
int32_t orc_score_groups(const orc_config *cfg, const orc_store *st,
                         int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                         const void *Q, int32_t T_q, int64_t q_stride_layer,
                         int64_t q_stride_head, int64_t q_stride_token,
                         float *scores, int32_t n_threads) {
    if (!check_cfg(cfg) || !st || !Q || !scores || T_q < 1) return ORC_ERR_ARG;
    if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > cfg->n_layers) return ORC_ERR_ARG;
    if (n_groups < 0 || n_groups > cfg->capacity_groups) return ORC_ERR_ARG;
    const int H = cfg->n_kv_heads, d = cfg->head_dim;
    const double eps = 1e-12;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
    for (int li = 0; li < layer_count; ++li) {
        const int l = layer_begin + li;
        double *q = (double *)malloc(sizeof(double) * (size_t)H * d);
        if (!q) return ORC_ERR_ARG;
        orc_query_embedding(cfg, Q, cfg->kv_dtype, (int64_t)li * q_stride_layer, T_q, q_stride_head, q_stride_token, q);
#pragma omp parallel for schedule(static)
        for (int t = 0; t < n_groups; ++t) {
            const float *kb = st->rep_key + meta_off(cfg, l, t, 0);
            if (cfg->score_mode == ORC_PER_LAYER) {
                double dot = 0.0, qn = 0.0, kn = 0.0;
                for (int i = 0; i < H * d; ++i) {
                    dot += q[i] * (double)kb[i];
                    qn += q[i] * q[i];
                    kn += (double)kb[i] * (double)kb[i];
                }
                double den = fmax(sqrt(qn), eps) * fmax(sqrt(kn), eps);
                scores[(int64_t)li * n_groups + t] = (float)(dot / den);
            } else {
                for (int h = 0; h < H; ++h) {
                    double dot = 0.0, qn = 0.0, kn = 0.0;
                    for (int c = 0; c < d; ++c) {
                        double qv = q[h * d + c], kv = (double)kb[h * d + c];
                        dot += qv * kv; qn += qv * qv; kn += kv * kv;
                    }
                    double den = fmax(sqrt(qn), eps) * fmax(sqrt(kn), eps);
                    scores[((int64_t)li * H + h) * n_groups + t] = (float)(dot / den);
                }
            }
        }
        free(q);
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* A3  top-K (appendix: K = min(ceil(B/G), T/G); indices kept sorted)   */
/* ------------------------------------------------------------------ */

int32_t orc_budget_to_k(int64_t budget_tokens, int32_t G, int32_t stored_groups) {
    int64_t k = (budget_tokens + G - 1) / G;
    return (int32_t)(k < stored_groups ? k : stored_groups);
}

typedef struct { float score; int32_t idx; } orc_pair;

static int cmp_score_desc_idx_asc(const void *a, const void *b) {
    const orc_pair *x = (const orc_pair *)a, *y = (const orc_pair *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}
static int cmp_idx_asc(const void *a, const void *b) {
    const orc_pair *x = (const orc_pair *)a, *y = (const orc_pair *)b;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/*
 * For each row: the min(k, n) largest scores (ties: lower index first), then
 * those indices in ascending order.  Unused slots of idx_out are -1 (their
 * score_out is 0).  n_sel_out[row] = min(k, n).
 */
int32_t orc_topk(const float *scores, int32_t rows, int32_t n, int64_t row_stride, int32_t k,
                 int32_t *idx_out, float *score_out, int32_t *n_sel_out) {
    if (!scores || !idx_out || rows < 0 || n < 0 || k < 1) return ORC_ERR_ARG;
    const int ksel = k < n ? k : n;
    for (int r = 0; r < rows; ++r) {
        orc_pair *p = (orc_pair *)malloc(sizeof(orc_pair) * (size_t)(n > 0 ? n : 1));
        if (!p) return ORC_ERR_ARG;
        for (int i = 0; i < n; ++i) { p[i].score = scores[(int64_t)r * row_stride + i]; p[i].idx = i; }
        qsort(p, (size_t)n, sizeof(orc_pair), cmp_score_desc_idx_asc);
        qsort(p, (size_t)ksel, sizeof(orc_pair), cmp_idx_asc);
        for (int j = 0; j < k; ++j) {
            idx_out[(int64_t)r * k + j] = j < ksel ? p[j].idx : -1;
            if (score_out) score_out[(int64_t)r * k + j] = j < ksel ? p[j].score : 0.0f;
        }
        if (n_sel_out) n_sel_out[r] = ksel;
        free(p);
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* A4  dequantize the selected groups into the active cache             */
/*     (Sec. 3.4 KV_active; appendix "Cache reconstruction")            */
/* ------------------------------------------------------------------ */

static void store_out(void *p, int64_t i, int dtype, float v) {
    if (dtype == ORC_BF16) ((uint16_t *)p)[i] = orc_f32_to_bf16(v);
    else if (dtype == ORC_FP16) ((uint16_t *)p)[i] = orc_f32_to_f16(v);
    else ((float *)p)[i] = v;
}

/*
 * idx: PER_LAYER -> [layer_count][k]; PER_HEAD -> [layer_count][H_k][k].
 * Slot j of a row lands at tokens token_offset + j*G .. + G-1 of the active
 * cache; element (l, h, tok, c) of k_active / v_active is at
 * (l-layer_begin)*stride_layer + h*stride_head + tok*stride_token + c.
 * Entries equal to -1 are skipped (their slot is left untouched).
 */
int32_t orc_dequant_gather(const orc_config *cfg, const orc_store *st,
                           int32_t layer_begin, int32_t layer_count,
                           const int32_t *idx, int32_t k, int32_t n_groups,
                           void *k_active, void *v_active, int32_t out_dtype,
                           int64_t stride_layer, int64_t stride_head, int64_t stride_token,
                           int32_t token_offset, int32_t n_threads) {
    if (!check_cfg(cfg) || !st || !idx || !k_active || !v_active || k < 1) return ORC_ERR_ARG;
    if (layer_begin < 0 || layer_count < 0 || layer_begin + layer_count > cfg->n_layers) return ORC_ERR_ARG;
    const int H = cfg->n_kv_heads, G = cfg->group_tokens, d = cfg->head_dim;
    const int per_head = cfg->score_mode == ORC_PER_HEAD;
    const int64_t nidx = (int64_t)layer_count * (per_head ? H : 1) * k;
    for (int64_t i = 0; i < nidx; ++i)
        if (idx[i] < -1 || idx[i] >= n_groups) return ORC_ERR_ARG;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
    const int64_t units = (int64_t)layer_count * k;
#pragma omp parallel for schedule(static)
    for (int64_t u = 0; u < units; ++u) {
        const int li = (int)(u / k), j = (int)(u % k), l = layer_begin + li;
        uint8_t *row = (uint8_t *)malloc((size_t)d);
        for (int h = 0; h < H; ++h) {
            const int t = per_head ? idx[((int64_t)li * H + h) * k + j] : idx[(int64_t)li * k + j];
            if (t < 0) continue;
            for (int which = 0; which < 2; ++which) {
                const uint8_t *codes = (which ? st->codes_v : st->codes_k) + codes_off(cfg, l, t, h);
                const float *s = (which ? st->scale_v : st->scale_k) + meta_off(cfg, l, t, h);
                const float *m = (which ? st->zero_v : st->zero_k) + meta_off(cfg, l, t, h);
                void *out = which ? v_active : k_active;
                for (int g = 0; g < G; ++g) {
                    orc_unpack_row(codes + (int64_t)g * code_row_bytes(cfg), d, cfg->bits, row);
                    int64_t base = (int64_t)li * stride_layer + (int64_t)h * stride_head +
                                   ((int64_t)token_offset + (int64_t)j * G + g) * stride_token;
                    for (int c = 0; c < d; ++c)
                        store_out(out, base + c, out_dtype, orc_dequant_value(row[c], s[c], m[c]));
                }
            }
        }
        free(row);
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* A5  decode attention over [system tokens || selected groups]         */
/*     (Sec. 3.4: decoding attends to the bounded active kv)            */
/* ------------------------------------------------------------------ */

/*
 * One layer.  q_dec [H_q][d] (dtype q_dtype).  Keys/values are the active
 * cache as orc_dequant_gather leaves it: element (h, tok, c) at
 * h*stride_head + tok*stride_token + c, n_tokens tokens, dtype kv_dtype
 * (values already rounded to that type, as the materialised cache holds
 * them).  out [H_q][d] rounded to out_dtype.  Plain softmax(q k^T * scale) v
 * in binary64.
 */
int32_t orc_attend(int32_t H_q, int32_t H_k, int32_t d, const void *q_dec, int32_t q_dtype,
                   const void *k_cache, const void *v_cache, int32_t kv_dtype,
                   int64_t stride_head, int64_t stride_token, int32_t n_tokens,
                   double softmax_scale, void *out, int32_t out_dtype) {
    if (H_q < 1 || H_k < 1 || H_q % H_k || d < 1 || n_tokens < 1) return ORC_ERR_ARG;
    const int rep = H_q / H_k;
    double *p = (double *)malloc(sizeof(double) * (size_t)n_tokens);
    double *acc = (double *)malloc(sizeof(double) * (size_t)d);
    if (!p || !acc) { free(p); free(acc); return ORC_ERR_ARG; }
    for (int hq = 0; hq < H_q; ++hq) {
        const int h = hq / rep;
        double mx = -INFINITY;
        for (int t = 0; t < n_tokens; ++t) {
            double dot = 0.0;
            for (int c = 0; c < d; ++c)
                dot += (double)load_elem(q_dec, (int64_t)hq * d + c, q_dtype) *
                       (double)load_elem(k_cache, h * stride_head + t * stride_token + c, kv_dtype);
            p[t] = dot * softmax_scale;
            if (p[t] > mx) mx = p[t];
        }
        double den = 0.0;
        for (int t = 0; t < n_tokens; ++t) { p[t] = exp(p[t] - mx); den += p[t]; }
        for (int c = 0; c < d; ++c) acc[c] = 0.0;
        for (int t = 0; t < n_tokens; ++t)
            for (int c = 0; c < d; ++c)
                acc[c] += p[t] * (double)load_elem(v_cache, h * stride_head + t * stride_token + c, kv_dtype);
        for (int c = 0; c < d; ++c) store_out(out, (int64_t)hq * d + c, out_dtype, (float)(acc[c] / den));
    }
    free(p); free(acc);
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* CTR (Sec. 3.3): temporal similarity, static / dynamic split, budget, */
/*     saliency selection of the dynamic tokens                         */
/* ------------------------------------------------------------------ */

/*
 * s_t^(i) = F_t^(i) . F_{t-1}^(i) / (|F_t^(i)| |F_{t-1}^(i)|)  for the frames t of one call.
 * F: element (t, i, c) at t*stride_frame + i*stride_token + c, T frames of N tokens of D channels.
 * prev (nullable): the features of the frame before F[0], [N][D] with the same token stride -- the state the
 * method carries from call to call; without it frame 0 has no predecessor and gets -inf.
 * sim: [T][N] binary32 (the binary64 result rounded once).
 */
int32_t orc_ctr_similarity(const void *F, const void *prev, int dtype, int32_t T, int32_t N, int32_t D,
                           int64_t stride_frame, int64_t stride_token, float *sim) {
    if (!F || !sim || T < 0 || N < 1 || D < 1) return ORC_ERR_ARG;
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < N; ++i) {
            const void *a_base = F, *b_base = F;
            int64_t a0 = (int64_t)t * stride_frame + (int64_t)i * stride_token, b0;
            if (t == 0) {
                if (!prev) { sim[(int64_t)t * N + i] = -INFINITY; continue; }
                b_base = prev;
                b0 = (int64_t)i * stride_token;
            } else {
                b0 = (int64_t)(t - 1) * stride_frame + (int64_t)i * stride_token;
            }
            double dot = 0.0, na = 0.0, nb = 0.0;
            for (int c = 0; c < D; ++c) {
                double a = (double)load_elem(a_base, a0 + c, dtype), b = (double)load_elem(b_base, b0 + c, dtype);
                dot += a * b;
                na += a * a;
                nb += b * b;
            }
            double da = sqrt(na), db = sqrt(nb);
            if (da < 1e-12) da = 1e-12;
            if (db < 1e-12) db = 1e-12;
            sim[(int64_t)t * N + i] = (float)(dot / (da * db));
        }
    return ORC_OK;
}

/*
 * Per frame: S_t = {i : s_t^(i) > tau_c}, D_t the rest; k_s = floor(G |S_t| / N), k_d = G - k_s;
 * G_d = the k_d dynamic tokens of largest saliency alpha.
 * static_idx [T][N]: S_t ascending, then -1.  dyn_idx [T][G]: G_d ascending, then -1.
 * k_s, k_d: [T].  (The k_s tokens that Merge would add are not produced here.)
 */
int32_t orc_ctr_select(const float *sim, const float *alpha, int32_t T, int32_t N, int32_t G, float tau_c,
                       int32_t *k_s, int32_t *k_d, int32_t *static_idx, int32_t *dyn_idx) {
    if (!sim || !alpha || !k_s || !k_d || !static_idx || !dyn_idx || T < 0 || N < 1 || G < 1 || G > N) return ORC_ERR_ARG;
    int32_t *dyn = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    uint8_t *taken = (uint8_t *)malloc((size_t)N);
    if (!dyn || !taken) { free(dyn); free(taken); return ORC_ERR_ARG; }
    for (int t = 0; t < T; ++t) {
        const float *s = sim + (int64_t)t * N, *a = alpha + (int64_t)t * N;
        int ns = 0, nd = 0;
        for (int i = 0; i < N; ++i) {
            if (s[i] > tau_c) static_idx[(int64_t)t * N + ns++] = i;
            else dyn[nd++] = i;
        }
        for (int i = ns; i < N; ++i) static_idx[(int64_t)t * N + i] = -1;
        const int ks = (int)(((int64_t)G * ns) / N), kd = G - ks;
        k_s[t] = ks;
        k_d[t] = kd;
        /* kd times: the not yet taken dynamic token of largest alpha, the lowest index among equals */
        memset(taken, 0, (size_t)N);
        int got = 0;
        for (int r = 0; r < kd && r < nd; ++r) {
            int best = -1;
            for (int j = 0; j < nd; ++j) {
                int i = dyn[j];
                if (taken[i]) continue;
                if (best < 0 || a[i] > a[best]) best = i; /* dyn is ascending: equal alpha keeps the earlier one */
            }
            if (best < 0) break; /* cannot happen while r < nd; keeps the index provably in range */
            taken[best] = 1;
            ++got;
        }
        int w = 0;
        for (int i = 0; i < N; ++i)
            if (taken[i]) dyn_idx[(int64_t)t * G + w++] = i;
        for (; w < G; ++w) dyn_idx[(int64_t)t * G + w] = -1;
        (void)got;
    }
    free(dyn);
    free(taken);
    return ORC_OK;
}

/*
 * Sec. 3.3, the Merge_{k_s} half of the (G_d, G_s) equation: the static tokens of one frame are consolidated into
 * k_s tokens by a density-based clustering.  The paper names the method (density peaks, going by its overview
 * figure) and fixes none of its parameters; the reading taken here -- the k-nearest-neighbour form of density-peak
 * clustering that token-merging work commonly uses -- is a decision of this code, written out step by step:
 *   d2(i,j) = sum_c (x_ic - x_jc)^2 / D                            squared distance, normalised by the width
 *   rho_i   = exp(-(1/kk) sum of the kk smallest d2(i,j), j != i)   kk = min(knn, n_s - 1); kk = 0 gives rho = 1
 *   delta_i = min d(i,j) over the j that are denser than i (rho_j > rho_i, or equal and j earlier), d = sqrt(d2);
 *             the densest token of all takes max_j d(i,j)
 *   gamma_i = rho_i * delta_i; the k_s tokens of largest gamma are the cluster centres (equal gammas: the earlier one)
 *   every other static token joins the centre it is nearest to (equal distances: the earlier centre)
 *   a cluster becomes one token: the arithmetic mean of its members' features, placed at its centre's position
 * F: one frame [N][D] of `dtype` (element (i, c) at i * stride_token + c); S: the n_s static token indices, ascending.
 * centre [k_s]: token indices of the centres, ascending; assign [n_s]: for every static token the position of its
 * centre in centre[]; merged [k_s][D]: the means (binary64 sums, returned in binary32); gamma [n_s] (nullable).
 * margin (nullable, 1 + n_s values): how far the integer decisions are from flipping -- [0] the relative gap between
 * the smallest gamma taken and the largest left out, [1 + a] the relative gap between static token a's nearest and
 * second nearest centre (+inf where there is nothing to compare: a centre, or a single cluster).
 */
int32_t orc_ctr_merge(const void *F, int32_t dtype, int32_t N, int32_t D, int64_t stride_token, const int32_t *S,
                      int32_t n_s, int32_t k_s, int32_t knn, int32_t *centre, int32_t *assign, float *merged,
                      double *gamma, double *margin) {
    if (!F || !S || !centre || !assign || !merged || N < 1 || D < 1 || n_s < 0 || n_s > N || k_s < 0 || k_s > n_s || knn < 0)
        return ORC_ERR_ARG;
    if (margin)
        for (int a = 0; a <= n_s; ++a) margin[a] = INFINITY;
    if (k_s == 0) return ORC_OK;
    for (int a = 0; a < n_s; ++a)
        if (S[a] < 0 || S[a] >= N || (a > 0 && S[a] <= S[a - 1])) return ORC_ERR_ARG;
    const size_t n = (size_t)n_s;
    double *d2 = (double *)malloc(sizeof(double) * n * n), *rho = (double *)malloc(sizeof(double) * n);
    double *gam = (double *)malloc(sizeof(double) * n), *tmp = (double *)malloc(sizeof(double) * n);
    uint8_t *is_c = (uint8_t *)calloc(n, 1);
    if (!d2 || !rho || !gam || !tmp || !is_c) { free(d2); free(rho); free(gam); free(tmp); free(is_c); return ORC_ERR_ARG; }
    for (int a = 0; a < n_s; ++a)
        for (int b = 0; b < n_s; ++b) {
            double acc = 0.0;
            for (int c = 0; c < D; ++c) {
                const double u = (double)load_elem(F, (int64_t)S[a] * stride_token + c, dtype) -
                                 (double)load_elem(F, (int64_t)S[b] * stride_token + c, dtype);
                acc += u * u;
            }
            d2[a * n + b] = acc / (double)D;
        }
    const int kk = knn < n_s - 1 ? knn : n_s - 1;
    for (int a = 0; a < n_s; ++a) {
        /* the kk smallest distances to OTHER tokens: selection by repeated minimum */
        int m = 0;
        for (int b = 0; b < n_s; ++b)
            if (b != a) tmp[m++] = d2[a * n + b];
        double sum = 0.0;
        for (int r = 0; r < kk; ++r) {
            int best = r;
            for (int j = r + 1; j < m; ++j)
                if (tmp[j] < tmp[best]) best = j;
            const double v = tmp[best];
            tmp[best] = tmp[r];
            tmp[r] = v;
            sum += v;
        }
        rho[a] = kk > 0 ? exp(-sum / (double)kk) : 1.0;
    }
    for (int a = 0; a < n_s; ++a) {
        double best = INFINITY, far = 0.0;
        for (int b = 0; b < n_s; ++b) {
            if (b == a) continue;
            const double d = sqrt(d2[a * n + b]);
            if (d > far) far = d;
            if ((rho[b] > rho[a] || (rho[b] == rho[a] && b < a)) && d < best) best = d;
        }
        gam[a] = rho[a] * (best == INFINITY ? far : best);
        if (gamma) gamma[a] = gam[a];
    }
    /* k_s times: the not yet taken token of largest gamma, the earliest among equals */
    double last_taken = INFINITY;
    for (int r = 0; r < k_s; ++r) {
        int best = -1;
        for (int a = 0; a < n_s; ++a)
            if (!is_c[a] && (best < 0 || gam[a] > gam[best])) best = a;
        is_c[best] = 1;
        last_taken = gam[best];
    }
    if (margin && k_s < n_s) {
        double next = -INFINITY;
        for (int a = 0; a < n_s; ++a)
            if (!is_c[a] && gam[a] > next) next = gam[a];
        margin[0] = (last_taken - next) / (fabs(last_taken) > 1e-300 ? fabs(last_taken) : 1e-300);
    }
    int w = 0;
    for (int a = 0; a < n_s; ++a)
        if (is_c[a]) centre[w++] = S[a];
    /* position of every centre among the static tokens, in centre order */
    int *cpos = (int *)malloc(sizeof(int) * (size_t)k_s);
    if (!cpos) { free(d2); free(rho); free(gam); free(tmp); free(is_c); return ORC_ERR_ARG; }
    w = 0;
    for (int a = 0; a < n_s; ++a)
        if (is_c[a]) cpos[w++] = a;
    for (int a = 0; a < n_s; ++a) {
        int best = 0;
        double second = INFINITY;
        if (is_c[a]) {
            for (int j = 0; j < k_s; ++j)
                if (cpos[j] == a) best = j;
        } else {
            for (int j = 1; j < k_s; ++j)
                if (d2[a * n + cpos[j]] < d2[a * n + cpos[best]]) best = j;
            for (int j = 0; j < k_s; ++j)
                if (j != best && d2[a * n + cpos[j]] < second) second = d2[a * n + cpos[j]];
            if (margin && k_s > 1) {
                const double near = d2[a * n + cpos[best]];
                margin[1 + a] = (second - near) / (second > 1e-300 ? second : 1e-300);
            }
        }
        assign[a] = best;
    }
    for (int j = 0; j < k_s; ++j)
        for (int c = 0; c < D; ++c) {
            double acc = 0.0;
            int cnt = 0;
            for (int a = 0; a < n_s; ++a)
                if (assign[a] == j) {
                    acc += (double)load_elem(F, (int64_t)S[a] * stride_token + c, dtype);
                    ++cnt;
                }
            merged[(int64_t)j * D + c] = (float)(acc / (double)cnt);
        }
    free(d2); free(rho); free(gam); free(tmp); free(is_c); free(cpos);
    return ORC_OK;
}

/*
 * Sec. 3.3, the retained group G_t of a frame (both paths together, |G_t| = G).  The k_d selected dynamic tokens
 * (their feature rows, unchanged) and the k_s merged tokens (rounded to the feature type, nearest-even), in ascending
 * order of token position -- a merged token stands at its centre's position.  retained [G][D] of `dtype`,
 * pos [G]; rows behind the k_d + k_s tokens are zero with position -1.
 */
int32_t orc_ctr_retain(const void *F, int32_t dtype, int32_t N, int32_t D, int64_t stride_token, const int32_t *dyn,
                       int32_t k_d, const int32_t *centre, const float *merged, int32_t k_s, int32_t G, void *retained,
                       int32_t *pos) {
    if (!F || !retained || !pos || k_d < 0 || k_s < 0 || k_d + k_s > G || D < 1 || N < 1) return ORC_ERR_ARG;
    int a = 0, b = 0;
    for (int w = 0; w < G; ++w) {
        const int pa = a < k_d ? dyn[a] : N + 1, pb = b < k_s ? centre[b] : N + 1;
        if (pa > N && pb > N) {
            pos[w] = -1;
            for (int c = 0; c < D; ++c) store_out(retained, (int64_t)w * D + c, dtype, 0.0f);
        } else if (pa < pb) {
            pos[w] = pa;
            for (int c = 0; c < D; ++c) store_out(retained, (int64_t)w * D + c, dtype, load_elem(F, (int64_t)pa * stride_token + c, dtype));
            ++a;
        } else {
            pos[w] = pb;
            for (int c = 0; c < D; ++c) store_out(retained, (int64_t)w * D + c, dtype, merged[(int64_t)b * D + c]);
            ++b;
        }
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* O8  storage accounting                                               */
/* ------------------------------------------------------------------ */

/* Sec. 3.2 / Sec. 3.4: (N*d*16 bits) / (G*d*bits) = 16N / (bits*G); 4N/G at 4 bits */
double orc_paper_ratio(int32_t N, int32_t G, int32_t bits) { return (16.0 * N) / ((double)bits * G); }

/* ablation table "Ratio (%)": stored bits relative to N tokens at 16 bit */
double orc_ratio_percent(int32_t N, int32_t G, int32_t bits) { return 100.0 * ((double)G * bits) / (16.0 * N); }

/* Sec. 3.1 growth equation integrated: 2 (K and V) * L * frames * N * H_kv * d_h * sizeof */
double orc_fp16_kv_bytes(int32_t L, int64_t frames, int32_t N, int32_t H_kv, int32_t d_h, int32_t elem_bytes) {
    return 2.0 * L * (double)frames * N * H_kv * d_h * elem_bytes;
}

/* bytes this store really holds for `groups` groups per layer, metadata included */
double orc_store_bytes(const orc_config *c, int64_t groups, int32_t with_metadata) {
    double per_head_codes = 2.0 * c->group_tokens * (double)code_row_bytes(c); /* K and V */
    double eb = c->meta_dtype == ORC_FP32 ? 4.0 : 2.0; /* bytes of one stored s, m or k-bar value */
    double per_head_meta = 4.0 * c->head_dim * eb /* sK mK sV mV */ + c->head_dim * eb /* k-bar */ + 4.0 /* norm */;
    double per = per_head_codes + (with_metadata ? per_head_meta : 0.0);
    return per * c->n_kv_heads * (double)groups * c->n_layers;
}

int32_t orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
