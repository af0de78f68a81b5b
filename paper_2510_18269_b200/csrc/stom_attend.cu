// A5: decode attention of one new query token over [system tokens || the
// selected groups], dequantizing the groups on the fly (paper Sec. 3.4:
// decoding attends to the bounded active kv, KV_active = union of the
// dequantized selected groups plus the full-precision system tokens; appendix
// "Cache reconstruction for decoding": the per-layer indices are reused for
// every decode step).  Nothing is materialised: a decode step reads the
// packed codes and their (s, m) -- a quarter of the bytes of the bf16 cache --
// instead of writing that cache once and re-reading it every step.
//
// Work unit: a segment = up to 32 consecutive tokens of one selected group (a
// group of 50 tokens is two segments) or of the system tokens.  A block of 8
// warps takes 8 consecutive segments of one (layer, kv head) and all the query
// heads of that kv head's GQA block (in chunks of 8); warp w owns segment w:
//   phase 1  scores of the segment's tokens against the query heads, a
//            tensor-core product whose matrix operand is the raw codes
//   phase 2  block-local softmax statistics per query head (max, sum) in the
//            base-2 domain (the scores carry softmax_scale * log2(e))
//   phase 3  weighted sum of V, again a tensor-core product over raw codes,
//            per warp; the warps' sums are combined through shared memory
// and writes (max, sum, weighted sum) per query head to the workspace.  The
// block that draws the last ticket of its (layer, kv head) merges the partial
// results of all its blocks and writes the output row.  Nobody waits.
// A decode step is latency, not bandwidth: 2.2 MB per layer at the 7B geometry.
#include "stom_internal.cuh"

namespace stom {

constexpr int kAtWarps = 8;
constexpr int kAtThreads = kAtWarps * 32;
constexpr int kAtSegTokens = 32;  // token slots per segment
constexpr int kAtHeads = 8;       // query heads handled together

struct AttendParams {
    const int32_t *idx;
    const uint8_t *codes_k, *codes_v;
    const void *scale_k, *zero_k, *scale_v, *zero_v;  // elements of g.meta_dtype
    const void *q;
    int64_t q_sl, q_sh;  // element strides of q_dec: layer, query head
    const void *ksys, *vsys;
    int64_t s_sl, s_sh, s_st;  // element strides of the system-token cache: layer, kv head, token
    void *out;
    int64_t o_sl, o_sh;  // element strides of out: layer, query head
    float *part;         // [layer][H][blocks][rep][d + 2]
    uint32_t *counters;  // [layer][H]
    BankGeom g;
    int32_t layer_begin, k, n_groups, per_head, rep, sys_len, n_sys_seg, n_seg, segs_per_group;
    float scale_log2e;
    uint32_t *flags;
};

// Ticket and merge, the tail of the attention kernel: every block of a (layer, kv head) has written its partial
// (max, sum, weighted sum) per query head to the workspace; the block that draws the last ticket combines them and
// writes the output rows.  All threads of the block call it; nobody waits for another block.
template <typename CT, int D>
__device__ __forceinline__ void attend_merge(const AttendParams &p, int li, int h, int n_blocks, int *s_last_ptr) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, H = p.g.H;
    int &s_last = *s_last_ptr;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned ticket = atomicAdd(&p.counters[li * H + h], 1u);
        // tickets of a cleared workspace run from 0 to n_blocks - 1; anything else was there before the call
        if (ticket >= (unsigned)n_blocks && p.flags) atomicOr(p.flags, STOM_FLAG_DIRTY_WORKSPACE);
        s_last = ticket == (unsigned)n_blocks - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) p.counters[li * H + h] = 0;  // as found
    // One warp per query head.  Lanes share out the blocks 32 at a time: (max, sum) of a block come in one 8-byte
    // load; the channel sums of the first kChunk blocks are requested in the same breath, before anything is
    // reduced, and those of the next chunk while the current one is added up -- the merge is two memory round trips
    // for up to kChunk blocks and one more per further chunk.
    constexpr int kChunk = D >= 256 ? 4 : 8;
    for (int hq = warp; hq < p.rep; hq += kAtWarps) {
        const float *rec0 = p.part + (((int64_t)li * H + h) * n_blocks * p.rep + hq) * (D + 2);
        const int64_t step = (int64_t)p.rep * (D + 2);
        auto load_chunk = [&](int b0, float (&v)[kChunk][D / 32]) {
#pragma unroll
            for (int j = 0; j < kChunk; ++j)
#pragma unroll
                for (int i = 0; i < D / 32; ++i)
                    v[j][i] = b0 + j < n_blocks ? __ldcg(rec0 + (b0 + j) * step + 2 + lane + 32 * i) : 0.0f;
        };
        float cur[kChunk][D / 32];
        load_chunk(0, cur);
        // the global maximum over all blocks (several trips only beyond 32 blocks)
        float2 ms = make_float2(-INFINITY, 0.0f);  // of block `lane` of the first trip
        if (lane < n_blocks) ms = __ldcg(reinterpret_cast<const float2 *>(rec0 + lane * step));
        float mx = ms.x;
        for (int b = lane + 32; b < n_blocks; b += 32) mx = fmaxf(mx, __ldcg(rec0 + b * step));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float den = 0.0f;
        float num[D / 32];
#pragma unroll
        for (int i = 0; i < D / 32; ++i) num[i] = 0.0f;
        for (int b0 = 0; b0 < n_blocks; b0 += 32) {
            if (b0 > 0) {
                ms = make_float2(-INFINITY, 0.0f);
                if (b0 + lane < n_blocks) ms = __ldcg(reinterpret_cast<const float2 *>(rec0 + (b0 + lane) * step));
            }
            const float w_mine = ms.x == -INFINITY ? 0.0f : exp2f(ms.x - mx);
            den = fmaf(ms.y, w_mine, den);
            const int nb = min(32, n_blocks - b0);
            for (int c0 = 0; c0 < nb; c0 += kChunk) {
                float nxt[kChunk][D / 32];
                const bool more = b0 + c0 + kChunk < n_blocks;
                if (more) load_chunk(b0 + c0 + kChunk, nxt);
#pragma unroll
                for (int j = 0; j < kChunk; ++j) {
                    const float w = __shfl_sync(0xffffffffu, w_mine, (c0 + j) & 31);
#pragma unroll
                    for (int i = 0; i < D / 32; ++i) num[i] = fmaf(cur[j][i], c0 + j < nb ? w : 0.0f, num[i]);
                }
                if (more) {
#pragma unroll
                    for (int j = 0; j < kChunk; ++j)
#pragma unroll
                        for (int i = 0; i < D / 32; ++i) cur[j][i] = nxt[j][i];
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
        CT *out = reinterpret_cast<CT *>(p.out) + (int64_t)li * p.o_sl + (int64_t)(h * p.rep + hq) * p.o_sh;
#pragma unroll
        for (int i = 0; i < D / 32; ++i) out[lane + 32 * i] = (CT)(den > 0.0f ? num[i] / den : 0.0f);
    }
}

// ---------------------------------------------------------------------------------------------------------------
// The two contractions on the tensor cores (4-bit and 2-bit codes).
//
// Both products are small dense contractions -- scores: [tokens x d] . [d x 8 query heads]; values:
// [d x tokens] . [tokens x 8 query heads] -- so they run as m16n8k16 warp-level matrix products (the query heads of a
// GQA block are the 8 columns).  The affine map of the quantizer is moved out of the inner product: within a group
// (s, m) depend on the channel only, so
//     scores:  sum_c q_c (code_c s_c + m_c) = sum_c code_c (q_c s_c) + sum_c q_c m_c
//     values:  sum_t w_t (code_tc s_c + m_c) = s_c sum_t w_t code_tc + m_c sum_t w_t
// and the matrix operand is the raw code.  A code becomes a bfloat16 without arithmetic: 0x4300 | code is the number
// 128 + code, exactly; the 128 is taken out again through the same sums.  The contraction index of a matrix product
// may be permuted freely as long as both operands use the same permutation, and so may the output columns: a thread
// therefore owns CONTIGUOUS code bytes (for the scores: d/4 adjacent channels of a token row; for the values: d/8
// adjacent channels of four tokens), which it loads with one vector load and slices with byte permutes.
// ---------------------------------------------------------------------------------------------------------------

template <typename MT>
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1);
template <>
__device__ __forceinline__ void mma_16816<__nv_bfloat16>(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <>
__device__ __forceinline__ void mma_16816<__half>(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

// NW 32-bit words from p (p aligned to min(16, 4 * NW) bytes), or zeros
template <int NW>
__device__ __forceinline__ void load_words_or_zero(const void *p, bool valid, uint32_t (&w)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = 0u;
    if (!valid) return;
    if constexpr (NW == 1) {
        w[0] = __ldg(static_cast<const uint32_t *>(p));
    } else if constexpr (NW == 2) {
        const uint2 v = __ldg(static_cast<const uint2 *>(p));
        w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
        for (int i = 0; i < NW / 4; ++i) {
            const uint4 v = __ldg(static_cast<const uint4 *>(p) + i);
            w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
        }
    }
}

// Field f of every byte of a word of packed codes (a byte holds 8/BITS codes, lowest channel in the lowest bits):
// byte b of the result is the code of channel (8/BITS) * b + f of the word, alone in its byte.
template <int BITS>
__device__ __forceinline__ uint32_t code_view(uint32_t w, int f) {
    return (w >> (BITS * f)) & (BITS == 4 ? 0x0F0F0F0Fu : 0x03030303u);
}
// Where code i of a run of packed codes sits: word, byte of the word, field of the byte.
template <int BITS> __device__ __forceinline__ constexpr int code_word_of(int i) { return i / (32 / BITS); }
template <int BITS> __device__ __forceinline__ constexpr int code_byte_of(int i) { return (i % (32 / BITS)) / (8 / BITS); }
template <int BITS> __device__ __forceinline__ constexpr int code_field_of(int i) { return i % (8 / BITS); }

// NB bytes of packed codes from p (aligned to min(16, NB) bytes) as 32-bit words, or zeros
template <int NB>
__device__ __forceinline__ void load_code_bytes(const uint8_t *p, bool valid, uint32_t (&w)[(NB + 3) / 4]) {
    if constexpr (NB == 2) {
        w[0] = valid ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(p)) : 0u;
    } else {
        load_words_or_zero<NB / 4>(p, valid, w);
    }
}

// Byte `b` of x and byte `b` of y, each holding one code (0x00..0x0F), as the bfloat16 pair
// (128 + code of x, 128 + code of y): the permute puts the two bytes into the low byte of each half and fills the
// other two with the sign of a source byte (selector values of 8 and above), which is zero.
__device__ __forceinline__ uint32_t code_pair_bf16(uint32_t x, uint32_t y, int b) {
    uint32_t v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(v) : "r"(x), "r"(y), "r"(0x8480u + (uint32_t)b * 0x0101u));
    return v | 0x43004300u;
}

// Two floats as a (high, low) pair of packed 16-bit pairs: hi = the values rounded to MT, lo = what the rounding
// left over, rounded again.  A matrix product issued once with each part carries 16 significant bits of the operand.
template <typename MT>
__device__ __forceinline__ void split2(float a, float b, uint32_t &hi, uint32_t &lo, float &seen_a, float &seen_b) {
    hi = pack2<MT>(a, b);
    float ha, hb, la, lb;
    unpack2<MT>(hi, ha, hb);
    lo = pack2<MT>(a - ha, b - hb);
    unpack2<MT>(lo, la, lb);
    seen_a = ha + la;
    seen_b = hb + lb;
}

// QT: type of q_dec; CT: type of the system-token cache and of the output; D: head dim; BITS: width of a code
template <typename QT, typename CT, int D, int BITS>
__global__ void __launch_bounds__(kAtThreads) attend_mma_kernel(const AttendParams p) {
    constexpr int kSlots = kAtWarps * kAtSegTokens;
    constexpr int kBuf = (32 * 1024) / (kAtHeads * D * 4) < kAtWarps ? (32 * 1024) / (kAtHeads * D * 4) : kAtWarps;
    constexpr int KS = D / 16;  // k-steps of the score product (16 channels each)
    constexpr int KC = D / 4;   // channels of a token row one thread owns in the score product
    constexpr int MT = D / 16;  // m-tiles of the value product (16 channels each)
    constexpr int VC = D / 8;   // channels one thread owns in the value product
    constexpr int KB = KC * BITS / 8, VB = VC * BITS / 8;  // bytes of packed codes behind them
    using BF = __nv_bfloat16;
    __shared__ __align__(16) float buf[8192];  // scores / weights [kAtHeads][kSlots]; then warp sums [kBuf][kAtHeads][D]
    __shared__ __align__(16) float qf[kAtHeads][D];
    __shared__ float blk_max[kAtHeads];
    __shared__ float seg_sum[kAtWarps][kAtHeads];  // sum of a segment's weights per query head, as the tensor core sees them
    __shared__ int s_last;
    static_assert(kAtHeads * kSlots <= 8192 && kBuf * kAtHeads * D <= 8192, "shared buffer");
    static_assert(kAtHeads == 8 && kAtSegTokens == 32, "fragment mapping");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;  // fragment coordinates of the thread
    const int bx = blockIdx.x, h = blockIdx.y, li = blockIdx.z;
    const int G = p.g.G, H = p.g.H;
    const int seg = bx * kAtWarps + warp;
    float(*sc)[kSlots] = reinterpret_cast<float(*)[kSlots]>(buf);

    // ---- what the warp's segment is
    int n_tok = 0, tok0 = 0;
    bool is_sys = false;
    int64_t slot = 0;
    if (seg < p.n_sys_seg) {
        is_sys = true;
        tok0 = seg * kAtSegTokens;
        n_tok = min(kAtSegTokens, p.sys_len - tok0);
    } else if (seg < p.n_seg) {
        const int sg = seg - p.n_sys_seg;
        const int j = sg / p.segs_per_group;
        tok0 = (sg - j * p.segs_per_group) * kAtSegTokens;
        const int tg = p.per_head ? p.idx[((int64_t)li * H + h) * p.k + j] : p.idx[(int64_t)li * p.k + j];
        if (tg >= 0 && tg < p.n_groups) {
            n_tok = min(kAtSegTokens, G - tok0);
            slot = bank_slot(p.g, p.layer_begin + li, tg, h);
        } else if (tg != -1 && p.flags && lane == 0 && tok0 == 0) {
            atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
        }
    }
    n_tok = max(n_tok, 0);
    const CT *ksys = reinterpret_cast<const CT *>(p.ksys) + (int64_t)li * p.s_sl + (int64_t)h * p.s_sh;
    const CT *vsys = reinterpret_cast<const CT *>(p.vsys) + (int64_t)li * p.s_sl + (int64_t)h * p.s_sh;
    const uint8_t *kcodes = p.codes_k + slot * (int64_t)G * p.g.row_bytes;
    const uint8_t *vcodes = p.codes_v + slot * (int64_t)G * p.g.row_bytes;
    const int md = p.g.meta_dtype;

    // A decode step is a chain of memory round trips.  Everything a group segment will read depends on the slot
    // only, not on the query: ask for it now (no registers are tied up), so that it arrives while the query rows are
    // staged and the loads below find it in L1.
    if (!is_sys && n_tok > 0) {
        const int esz = md == STOM_FP32 ? 4 : 2;
        const int64_t kat = (slot * D + KC * t) * esz, vat = (slot * D + VC * g) * esz;
        prefetch_l1(static_cast<const uint8_t *>(p.scale_k) + kat);
        prefetch_l1(static_cast<const uint8_t *>(p.zero_k) + kat);
        prefetch_l1(static_cast<const uint8_t *>(p.scale_v) + vat);
        prefetch_l1(static_cast<const uint8_t *>(p.zero_v) + vat);
#pragma unroll
        for (int i = 0; i < kAtSegTokens / 8; ++i) {
            const int row = g + 8 * i;  // the score product reads rows g, g+8, g+16, g+24
            if (row < n_tok) prefetch_l1(kcodes + (int64_t)(tok0 + row) * p.g.row_bytes + t * KB);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int tok = (i >> 2) * 16 + 2 * t + (i & 1) + 8 * ((i >> 1) & 1);  // the value product's tokens
            if (tok < n_tok) prefetch_l1(vcodes + (int64_t)(tok0 + tok) * p.g.row_bytes + g * VB);
        }
    }

    const int n_blocks = gridDim.x;
    for (int h0 = 0; h0 < p.rep; h0 += kAtHeads) {
        const int nh = min(kAtHeads, p.rep - h0);
        // ---- the query rows, scaled so that exp2 can be used
        for (int e = tid; e < kAtHeads * D; e += kAtThreads) {
            const int hh = e / D, c = e - hh * D;
            float v = 0.0f;
            if (hh < nh) {
                const QT *q = reinterpret_cast<const QT *>(p.q) + (int64_t)li * p.q_sl + (int64_t)(h * p.rep + h0 + hh) * p.q_sh;
                v = (float)q[c] * p.scale_log2e;
            }
            qf[hh][c] = v;
        }
        __syncthreads();

        // ---- phase 1: scores.  Contraction slot (kk; 2t, 2t+1, 2t+8, 2t+9) of the matrix product stands for
        //      channels KC*t + 4*kk + (0, 1, 2, 3); column g is query head g.
        for (int e = lane; e < kAtHeads * kAtSegTokens; e += 32)
            sc[e / kAtSegTokens][warp * kAtSegTokens + (e % kAtSegTokens)] = -INFINITY;  // slots without a token
        __syncwarp();
        if (n_tok > 0) {
            uint32_t qb[KS][2], ql[KS][2];  // the thread's column of the right-hand operand, high and low parts
            float bias = 0.0f;   // what the raw-code product leaves out, for query head g
            if (!is_sys) {
#pragma unroll
                for (int c8 = 0; c8 < KC / 8; ++c8) {
                    float s8[8], m8[8];
                    load_scale_zero8(p.scale_k, p.zero_k, slot * D + KC * t + c8 * 8, md, s8, m8);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {  // 2 channels each
                        const int c = KC * t + c8 * 8 + 2 * j;
                        const float q0 = qf[g][c], q1 = qf[g][c + 1];
                        uint32_t whi, wlo;
                        float r0, r1;  // the two products as the tensor core sees them
                        split2<BF>(q0 * s8[2 * j], q1 * s8[2 * j + 1], whi, wlo, r0, r1);
                        bias = fmaf(q0, m8[2 * j], bias);
                        bias = fmaf(q1, m8[2 * j + 1], bias);
                        bias = fmaf(-128.0f, r0 + r1, bias);
                        qb[(c8 * 8 + 2 * j) / 4][((c8 * 8 + 2 * j) / 2) & 1] = whi;
                        ql[(c8 * 8 + 2 * j) / 4][((c8 * 8 + 2 * j) / 2) & 1] = wlo;
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < KC / 2; ++j) {
                    const int c = KC * t + 2 * j;
                    float r0, r1;
                    split2<CT>(qf[g][c], qf[g][c + 1], qb[j / 2][j & 1], ql[j / 2][j & 1], r0, r1);
                }
            }
            bias += __shfl_xor_sync(0xffffffffu, bias, 1);
            bias += __shfl_xor_sync(0xffffffffu, bias, 2);
            const float bias_a = __shfl_sync(0xffffffffu, bias, (2 * t) << 2);       // of query head 2t
            const float bias_b = __shfl_sync(0xffffffffu, bias, (2 * t + 1) << 2);   // of query head 2t + 1
#pragma unroll
            for (int mt = 0; mt < kAtSegTokens / 16; ++mt) {
                const int r0 = mt * 16 + g, r1 = r0 + 8;
                if (mt * 16 >= n_tok) break;  // warp-uniform
                float c4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                if (!is_sys) {
                    uint32_t w0[(KB + 3) / 4], w1[(KB + 3) / 4];  // the thread's KC codes of the two token rows
                    load_code_bytes<KB>(kcodes + (int64_t)(tok0 + r0) * p.g.row_bytes + t * KB, r0 < n_tok, w0);
                    load_code_bytes<KB>(kcodes + (int64_t)(tok0 + r1) * p.g.row_bytes + t * KB, r1 < n_tok, w1);
#pragma unroll
                    for (int kk = 0; kk < KS; ++kk) {
                        // codes 4kk, 4kk+1 of the thread's run share a byte, and so do 4kk+2, 4kk+3
                        const int ca = 4 * kk, cb = 4 * kk + 2;
                        const int wa = code_word_of<BITS>(ca), ba = code_byte_of<BITS>(ca), fa = code_field_of<BITS>(ca);
                        const int wb = code_word_of<BITS>(cb), bb = code_byte_of<BITS>(cb), fb = code_field_of<BITS>(cb);
                        const uint32_t a0 = code_pair_bf16(code_view<BITS>(w0[wa], fa), code_view<BITS>(w0[wa], fa + 1), ba);
                        const uint32_t a1 = code_pair_bf16(code_view<BITS>(w1[wa], fa), code_view<BITS>(w1[wa], fa + 1), ba);
                        const uint32_t a2 = code_pair_bf16(code_view<BITS>(w0[wb], fb), code_view<BITS>(w0[wb], fb + 1), bb);
                        const uint32_t a3 = code_pair_bf16(code_view<BITS>(w1[wb], fb), code_view<BITS>(w1[wb], fb + 1), bb);
                        mma_16816<BF>(c4, a0, a1, a2, a3, qb[kk][0], qb[kk][1]);
                        mma_16816<BF>(c4, a0, a1, a2, a3, ql[kk][0], ql[kk][1]);
                    }
                } else {
                    uint32_t w0[KC / 2], w1[KC / 2];  // the thread's KC channels of the two token rows, 16-bit pairs
                    load_words_or_zero<KC / 2>(ksys + (int64_t)(tok0 + r0) * p.s_st + KC * t, r0 < n_tok, w0);
                    load_words_or_zero<KC / 2>(ksys + (int64_t)(tok0 + r1) * p.s_st + KC * t, r1 < n_tok, w1);
#pragma unroll
                    for (int kk = 0; kk < KS; ++kk) {
                        mma_16816<CT>(c4, w0[2 * kk], w1[2 * kk], w0[2 * kk + 1], w1[2 * kk + 1], qb[kk][0], qb[kk][1]);
                        mma_16816<CT>(c4, w0[2 * kk], w1[2 * kk], w0[2 * kk + 1], w1[2 * kk + 1], ql[kk][0], ql[kk][1]);
                    }
                }
                if (r0 < n_tok) {
                    sc[2 * t][warp * kAtSegTokens + r0] = c4[0] + bias_a;
                    sc[2 * t + 1][warp * kAtSegTokens + r0] = c4[1] + bias_b;
                }
                if (r1 < n_tok) {
                    sc[2 * t][warp * kAtSegTokens + r1] = c4[2] + bias_a;
                    sc[2 * t + 1][warp * kAtSegTokens + r1] = c4[3] + bias_b;
                }
            }
        }
        __syncthreads();

        // ---- phase 2: the block's maximum per query head; scores become weights in place.  The sum of the weights is
        //      taken in phase 3 from the ROUNDED weights the matrix product uses, so that numerator and denominator
        //      of the softmax average see the same weights.
        if (warp < kAtHeads) {
            float mx = -INFINITY;
            for (int i = lane; i < kSlots; i += 32) mx = fmaxf(mx, sc[warp][i]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            for (int i = lane; i < kSlots; i += 32) {
                const float v = sc[warp][i];
                sc[warp][i] = v == -INFINITY ? 0.0f : exp2f(v - mx);
            }
            if (lane == 0) blk_max[warp] = mx;
        }
        __syncthreads();

        // ---- phase 3: weighted sum of the values.  Rows of the product are channels: rows g and g + 8 of m-tile mm
        //      stand for channels VC*g + 2*mm and VC*g + 2*mm + 1; the contraction runs over the segment's tokens
        //      (slot 2t, 2t+1, 2t+8, 2t+9 of k-step ks is token 16*ks + the same); columns are query heads.
        float acc[MT][4];
#pragma unroll
        for (int mm = 0; mm < MT; ++mm)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mm][i] = 0.0f;
        float wsum = 0.0f;  // sum of the weights of query head g as the tensor core sees them
        if (n_tok > 0) {
#pragma unroll
            for (int ks = 0; ks < kAtSegTokens / 16; ++ks) {
                if (ks * 16 >= n_tok) break;  // warp-uniform
                const int ta = ks * 16 + 2 * t;  // tokens ta, ta + 1, ta + 8, ta + 9
                const float2 wlo = *reinterpret_cast<const float2 *>(&sc[g][warp * kAtSegTokens + ta]);
                const float2 whi = *reinterpret_cast<const float2 *>(&sc[g][warp * kAtSegTokens + ta + 8]);
                uint32_t b0, b1, l0, l1;  // the weights, high and low parts
                float r0, r1, r2, r3;
                if (!is_sys) {
                    split2<BF>(wlo.x, wlo.y, b0, l0, r0, r1);
                    split2<BF>(whi.x, whi.y, b1, l1, r2, r3);
                } else {
                    split2<CT>(wlo.x, wlo.y, b0, l0, r0, r1);
                    split2<CT>(whi.x, whi.y, b1, l1, r2, r3);
                }
                wsum += (r0 + r1) + (r2 + r3);
                if (!is_sys) {
                    uint32_t w[4][(VB + 3) / 4];  // the thread's VC codes of its 4 tokens
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tok = ta + (i & 1) + 8 * (i >> 1);
                        load_code_bytes<VB>(vcodes + (int64_t)(tok0 + tok) * p.g.row_bytes + g * VB, tok < n_tok, w[i]);
                    }
#pragma unroll
                    for (int mm = 0; mm < MT; ++mm) {
                        // channels VC*g + 2*mm and the next one share a byte; rows g and g + 8 of the m-tile
                        const int c = 2 * mm;
                        const int j = code_word_of<BITS>(c), b = code_byte_of<BITS>(c), f = code_field_of<BITS>(c);
                        const uint32_t a0 = code_pair_bf16(code_view<BITS>(w[0][j], f), code_view<BITS>(w[1][j], f), b);
                        const uint32_t a1 = code_pair_bf16(code_view<BITS>(w[0][j], f + 1), code_view<BITS>(w[1][j], f + 1), b);
                        const uint32_t a2 = code_pair_bf16(code_view<BITS>(w[2][j], f), code_view<BITS>(w[3][j], f), b);
                        const uint32_t a3 = code_pair_bf16(code_view<BITS>(w[2][j], f + 1), code_view<BITS>(w[3][j], f + 1), b);
                        mma_16816<BF>(acc[mm], a0, a1, a2, a3, b0, b1);
                        mma_16816<BF>(acc[mm], a0, a1, a2, a3, l0, l1);
                    }
                } else {
                    uint32_t w[4][VC / 2];  // the thread's VC channels of its 4 tokens, 16-bit pairs (channel 2mm, 2mm+1)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int tok = ta + (i & 1) + 8 * (i >> 1);
                        load_words_or_zero<VC / 2>(vsys + (int64_t)(tok0 + tok) * p.s_st + VC * g, tok < n_tok, w[i]);
                    }
#pragma unroll
                    for (int mm = 0; mm < MT; ++mm) {
                        const uint32_t a0 = __byte_perm(w[0][mm], w[1][mm], 0x5410), a1 = __byte_perm(w[0][mm], w[1][mm], 0x7632);
                        const uint32_t a2 = __byte_perm(w[2][mm], w[3][mm], 0x5410), a3 = __byte_perm(w[2][mm], w[3][mm], 0x7632);
                        mma_16816<CT>(acc[mm], a0, a1, a2, a3, b0, b1);
                        mma_16816<CT>(acc[mm], a0, a1, a2, a3, l0, l1);
                    }
                }
            }
        }
        wsum += __shfl_xor_sync(0xffffffffu, wsum, 1);
        wsum += __shfl_xor_sync(0xffffffffu, wsum, 2);
        const float ws_a = __shfl_sync(0xffffffffu, wsum, (2 * t) << 2), ws_b = __shfl_sync(0xffffffffu, wsum, (2 * t + 1) << 2);
        if (t == 0) seg_sum[warp][g] = wsum;
        if (!is_sys && n_tok > 0) {
            // acc holds sum_t w_t (128 + code): apply the group's scale and offset, channel by channel
#pragma unroll
            for (int c8 = 0; c8 < VC / 8; ++c8) {
                float s8[8], m8[8];
                load_scale_zero8(p.scale_v, p.zero_v, slot * D + VC * g + c8 * 8, md, s8, m8);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int mm = c8 * 4 + j;
                    acc[mm][0] = fmaf(s8[2 * j], fmaf(-128.0f, ws_a, acc[mm][0]), m8[2 * j] * ws_a);
                    acc[mm][1] = fmaf(s8[2 * j], fmaf(-128.0f, ws_b, acc[mm][1]), m8[2 * j] * ws_b);
                    acc[mm][2] = fmaf(s8[2 * j + 1], fmaf(-128.0f, ws_a, acc[mm][2]), m8[2 * j + 1] * ws_a);
                    acc[mm][3] = fmaf(s8[2 * j + 1], fmaf(-128.0f, ws_b, acc[mm][3]), m8[2 * j + 1] * ws_b);
                }
            }
        }
        __syncthreads();  // every warp is done with the weights; the buffer now takes the warps' sums
        float tot[kAtHeads * D / kAtThreads];
#pragma unroll
        for (int e = 0; e < kAtHeads * D / kAtThreads; ++e) tot[e] = 0.0f;
        for (int r = 0; r < kAtWarps; r += kBuf) {
            if (warp >= r && warp < r + kBuf) {
                float *dst = buf + (size_t)(warp - r) * kAtHeads * D;
#pragma unroll
                for (int mm = 0; mm < MT; ++mm) {
                    const int c = VC * g + 2 * mm;
                    dst[(2 * t) * D + c] = acc[mm][0];
                    dst[(2 * t + 1) * D + c] = acc[mm][1];
                    dst[(2 * t) * D + c + 1] = acc[mm][2];
                    dst[(2 * t + 1) * D + c + 1] = acc[mm][3];
                }
            }
            __syncthreads();
#pragma unroll
            for (int e = 0; e < kAtHeads * D / kAtThreads; ++e) {
                const int i = e * kAtThreads + tid;  // (head, channel) pair
                for (int w = 0; w < kBuf && r + w < kAtWarps; ++w) tot[e] += buf[(size_t)w * kAtHeads * D + i];
            }
            __syncthreads();
        }
        // ---- partial result of this block: (max, sum, weighted sum) per query head
#pragma unroll
        for (int e = 0; e < kAtHeads * D / kAtThreads; ++e) {
            const int i = e * kAtThreads + tid, hh = i / D, c = i - hh * D;
            if (hh < nh) {
                float *rec = p.part + ((((int64_t)li * H + h) * n_blocks + bx) * p.rep + h0 + hh) * (D + 2);
                rec[2 + c] = tot[e];
                if (c == 0) {
                    float sum = 0.0f;
#pragma unroll
                    for (int w = 0; w < kAtWarps; ++w) sum += seg_sum[w][hh];
                    rec[0] = blk_max[hh];
                    rec[1] = sum;
                }
            }
        }
        __syncthreads();  // qf, buf and the statistics are rewritten by the next chunk of heads
    }
    attend_merge<CT, D>(p, li, h, n_blocks, &s_last);
}

// The ticket counters take the same room whatever the layer range of a call, so that a workspace cleared once serves
// calls over any layer range of the bank.
static int64_t attend_counter_bytes(const stom_oqm_config *cfg) {
    return ((int64_t)cfg->n_layers * cfg->n_kv_heads * 4 + 255) / 256 * 256;
}

static int attend_segments(const stom_oqm_config *cfg, int32_t k, int32_t sys_len, int *n_sys_seg, int *segs_per_group) {
    *n_sys_seg = (sys_len + kAtSegTokens - 1) / kAtSegTokens;
    *segs_per_group = (cfg->group_tokens + kAtSegTokens - 1) / kAtSegTokens;
    return *n_sys_seg + k * *segs_per_group;
}

template <typename QT, typename CT>
static int32_t launch_attend(const AttendParams &p, dim3 grid, cudaStream_t s) {
    const bool b4 = p.g.row_bytes * 2 == p.g.d;  // 4-bit codes: d/2 bytes per row
    switch (p.g.d) {
    case 64:
        if (b4) attend_mma_kernel<QT, CT, 64, 4><<<grid, kAtThreads, 0, s>>>(p);
        else attend_mma_kernel<QT, CT, 64, 2><<<grid, kAtThreads, 0, s>>>(p);
        break;
    case 128:
        if (b4) attend_mma_kernel<QT, CT, 128, 4><<<grid, kAtThreads, 0, s>>>(p);
        else attend_mma_kernel<QT, CT, 128, 2><<<grid, kAtThreads, 0, s>>>(p);
        break;
    case 256:
        if (b4) attend_mma_kernel<QT, CT, 256, 4><<<grid, kAtThreads, 0, s>>>(p);
        else attend_mma_kernel<QT, CT, 256, 2><<<grid, kAtThreads, 0, s>>>(p);
        break;
    default: return STOM_ERR_SHAPE;
    }
    return finish_launch();
}

}  // namespace stom

using namespace stom;

extern "C" int64_t stom_oqm_attend_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count, int32_t k,
                                                   int32_t sys_len) {
    if (check_config(cfg) || layer_count < 0 || k < 0 || sys_len < 0) return STOM_ERR_INVALID_ARG;
    int n_sys_seg = 0, spg = 0;
    const int n_seg = attend_segments(cfg, k, sys_len, &n_sys_seg, &spg);
    const int64_t blocks = (n_seg + kAtWarps - 1) / kAtWarps;
    const int64_t counters = attend_counter_bytes(cfg);
    const int64_t part = (int64_t)layer_count * cfg->n_kv_heads * blocks * (cfg->n_q_heads / cfg->n_kv_heads) *
                         (cfg->head_dim + 2) * 4;
    return counters + (part + 255) / 256 * 256;
}

extern "C" int32_t stom_oqm_attend(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                   int32_t layer_begin, int32_t layer_count,
                                   const int32_t *idx, int32_t k, int32_t n_groups,
                                   const void *q_dec, int64_t q_stride_layer, int64_t q_stride_head,
                                   const void *k_sys, const void *v_sys, int32_t cache_dtype,
                                   int64_t sys_stride_layer, int64_t sys_stride_head, int64_t sys_stride_token,
                                   int32_t sys_len, float softmax_scale,
                                   void *out, int64_t out_stride_layer, int64_t out_stride_head,
                                   void *workspace, int64_t workspace_bytes, uint32_t *dev_flags, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if ((rc = check_store(store))) return rc;
    if ((rc = check_layers(cfg, layer_begin, layer_count))) return rc;
    if (!q_dec || !out || k < 0 || n_groups < 0 || sys_len < 0 || (k > 0 && !idx)) return STOM_ERR_INVALID_ARG;
    if (k + sys_len < 1) return STOM_ERR_INVALID_ARG;
    if (sys_len > 0 && (!k_sys || !v_sys)) return STOM_ERR_INVALID_ARG;
    if (n_groups > cfg->capacity_groups) return STOM_ERR_CAPACITY;
    if (cache_dtype != STOM_BF16 && cache_dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    if (q_stride_layer < 0 || q_stride_head < cfg->head_dim || out_stride_layer < 0 || out_stride_head < cfg->head_dim ||
        sys_stride_layer < 0 || sys_stride_head < 0 || (sys_len > 0 && sys_stride_token < cfg->head_dim))
        return STOM_ERR_INVALID_ARG;
    if ((idx && (reinterpret_cast<uintptr_t>(idx) & 3u)) || (reinterpret_cast<uintptr_t>(q_dec) & 3u) ||
        (reinterpret_cast<uintptr_t>(out) & 1u))
        return STOM_ERR_ALIGNMENT;
    if (sys_len > 0 && (!aligned16(k_sys) || !aligned16(v_sys) || !stride_ok(sys_stride_layer, cache_dtype) ||
                        !stride_ok(sys_stride_head, cache_dtype) || !stride_ok(sys_stride_token, cache_dtype)))
        return STOM_ERR_ALIGNMENT;
    const int64_t need = stom_oqm_attend_workspace_bytes(cfg, layer_count, k, sys_len);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need) return STOM_ERR_WORKSPACE;
    if (layer_count == 0) return STOM_OK;

    AttendParams p;
    p.idx = idx;
    p.codes_k = store->codes_k; p.codes_v = store->codes_v;
    p.scale_k = store->scale_k; p.zero_k = store->zero_k; p.scale_v = store->scale_v; p.zero_v = store->zero_v;
    p.q = q_dec; p.q_sl = q_stride_layer; p.q_sh = q_stride_head;
    p.ksys = k_sys; p.vsys = v_sys; p.s_sl = sys_stride_layer; p.s_sh = sys_stride_head; p.s_st = sys_stride_token;
    p.out = out; p.o_sl = out_stride_layer; p.o_sh = out_stride_head;
    const int64_t counters = attend_counter_bytes(cfg);
    p.counters = static_cast<uint32_t *>(workspace);
    p.part = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + counters);
    p.g = bank_geom(cfg);
    p.layer_begin = layer_begin; p.k = k; p.n_groups = n_groups;
    p.per_head = cfg->score_mode == STOM_SCORE_PER_HEAD;
    p.rep = cfg->n_q_heads / cfg->n_kv_heads;
    p.sys_len = sys_len;
    p.n_seg = attend_segments(cfg, k, sys_len, &p.n_sys_seg, &p.segs_per_group);
    p.scale_log2e = softmax_scale * 1.4426950408889634f;
    p.flags = dev_flags;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The ticket counters at the head of the workspace are zero on entry (the caller cleared the workspace once) and
    // every call leaves them zero: no memset here -- ahead of the kernel in a CUDA graph it measured 7 us per call.
    if (layer_count > 65535 || cfg->n_kv_heads > 65535) return STOM_ERR_SHAPE;
    const dim3 grid((p.n_seg + kAtWarps - 1) / kAtWarps, cfg->n_kv_heads, layer_count);
    const bool bf = cache_dtype == STOM_BF16;
    switch (cfg->kv_dtype) {
    case STOM_BF16:
        return bf ? launch_attend<__nv_bfloat16, __nv_bfloat16>(p, grid, s) : launch_attend<__nv_bfloat16, __half>(p, grid, s);
    case STOM_FP16:
        return bf ? launch_attend<__half, __nv_bfloat16>(p, grid, s) : launch_attend<__half, __half>(p, grid, s);
    default:
        return bf ? launch_attend<float, __nv_bfloat16>(p, grid, s) : launch_attend<float, __half>(p, grid, s);
    }
}
