// A5: decode attention of one new query token over [system tokens || the
// selected groups], dequantizing the groups on the fly (paper Sec. 3.4:
// decoding attends to the bounded active kv, KV_active = union of the
// dequantized selected groups plus the full-precision system tokens; appendix
// "Cache reconstruction for decoding": the per-layer indices are reused for
// every decode step).  Nothing is materialised: a decode step reads the
// packed codes and their (s, m) -- a quarter of the bytes of the bf16 cache --
// instead of writing that cache once and re-reading it every step.
//
// Work unit: one selected group (its G tokens) or a run of up to 16 system
// tokens.  Everything a unit reads is contiguous in the bank -- the K codes and
// the V codes of a (layer, group, kv head) are one block each, and so are its
// four metadata rows -- so a unit arrives in shared memory by a handful of bulk
// asynchronous copies (cp.async.bulk, completion counted on an mbarrier),
// which tie up no registers and no warp while the bytes are on their way.
//
//   grid     (C, kv heads, layers); the C blocks of a (layer, kv head) form a
//            thread-block cluster and share out its units
//   warp     owns its own ring of 1 or 2 stages and its own units (u = rank +
//            C * (warp + 8 * i)): lane 0 posts the copies of unit i + stages
//            as soon as unit i has been consumed.  Per unit the warp computes
//            scores (a tensor-core product over the raw codes), a warp-local
//            online softmax, and the weighted sum of V (again a tensor-core
//            product over raw codes); it keeps a running (max, sum, output)
//            for the 8 query heads it handles, so no block barrier sits
//            between units
//   merge    the warps of a block combine through shared memory, the blocks
//            of the cluster through distributed shared memory (one hardware
//            cluster barrier on each side); rank r writes its share of the
//            output rows.  No workspace, no tickets, nobody spins.
#include "stom_async.cuh"
#include "stom_internal.cuh"

namespace stom {

constexpr int kAtWarps = 8;
constexpr int kAtThreads = kAtWarps * 32;
constexpr int kAtUnitTokens = 64;  // token slots of a group unit (G <= 64)
constexpr int kAtSysTokens = 16;   // tokens of a system-token unit
constexpr int kAtHeads = 8;        // query heads handled together
constexpr int kAtWPitch = 68;      // floats per head row of a warp's weight tile (64 token slots + padding)
constexpr int kAtMaxStages = 2;
constexpr unsigned long long kAtWaitLimitNs = 2000000000ull;  // a copy that has not landed after 2 s ends the block

// Shared-memory layout (bytes from the start of dynamic shared memory)
constexpr int kAtOffBars = 0;                                   // [kAtWarps][kAtMaxStages] mbarriers
constexpr int kAtOffAbort = kAtOffBars + kAtWarps * kAtMaxStages * 8;
constexpr int kAtOffStat = 256;                                 // [kAtWarps][16]: max[8], sum[8] of each warp
constexpr int kAtOffBlk = kAtOffStat + kAtWarps * 16 * 4;       // max[8], sum[8] of the block
constexpr int kAtOffWt = kAtOffBlk + 16 * 4;                    // [kAtWarps][8][kAtWPitch] weights
constexpr int kAtOffOb = kAtOffWt + kAtWarps * kAtHeads * kAtWPitch * 4;  // the block's partial output
__host__ __device__ constexpr int at_opitch(int D) { return D + 8; }      // floats of one channel slab (D/8 channels x 8 heads) + padding
__host__ __device__ constexpr int at_ofloats(int D) { return 8 * at_opitch(D); }
__host__ __device__ constexpr int at_off_ring(int D) { return (kAtOffOb + at_ofloats(D) * 4 + 127) / 128 * 128; }

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
    BankGeom g;
    int32_t layer_begin, k, n_groups, per_head, rep, sys_len, n_sys_units, n_units;
    int32_t stage_bytes, n_stages;
    float scale_log2e;
    uint32_t *flags;
};

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
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <>
__device__ __forceinline__ void mma_16816<__half>(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NW 32-bit words from shared memory at p (aligned to min(16, 4 * NW) bytes), or zeros
template <int NW>
__device__ __forceinline__ void lds_words_or_zero(const unsigned char *p, bool valid, uint32_t (&w)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = 0u;
    if (!valid) return;
    if constexpr (NW == 1) {
        w[0] = *reinterpret_cast<const uint32_t *>(p);
    } else if constexpr (NW == 2) {
        const uint2 v = *reinterpret_cast<const uint2 *>(p);
        w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
        for (int i = 0; i < NW / 4; ++i) {
            const uint4 v = *(reinterpret_cast<const uint4 *>(p) + i);
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

// NB bytes of packed codes from shared memory at p (aligned to min(16, NB) bytes) as 32-bit words, or zeros
template <int NB>
__device__ __forceinline__ void lds_code_bytes(const unsigned char *p, bool valid, uint32_t (&w)[(NB + 3) / 4]) {
    if constexpr (NB == 2) {
        w[0] = valid ? (uint32_t)*reinterpret_cast<const uint16_t *>(p) : 0u;
    } else {
        lds_words_or_zero<NB / 4>(p, valid, w);
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

// Eight adjacent metadata values (element type by the run-time code md) from shared memory, as floats
__device__ __forceinline__ void lds_meta8(const unsigned char *row, int ch, int md, float (&f)[8]) {
    if (md == STOM_FP32) {
        const float4 a = *reinterpret_cast<const float4 *>(row + ch * 4), b = *reinterpret_cast<const float4 *>(row + ch * 4 + 16);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    } else {
        const uint4 v = *reinterpret_cast<const uint4 *>(row + ch * 2);
        if (md == STOM_BF16) {
            unpack2<__nv_bfloat16>(v.x, f[0], f[1]); unpack2<__nv_bfloat16>(v.y, f[2], f[3]);
            unpack2<__nv_bfloat16>(v.z, f[4], f[5]); unpack2<__nv_bfloat16>(v.w, f[6], f[7]);
        } else {
            unpack2<__half>(v.x, f[0], f[1]); unpack2<__half>(v.y, f[2], f[3]);
            unpack2<__half>(v.z, f[4], f[5]); unpack2<__half>(v.w, f[6], f[7]);
        }
    }
}

// The thread's KC query channels, kept in registers in the type they arrive in
template <typename QT, int KC>
struct QRegs {
    static constexpr int W = sizeof(QT) == 4 ? KC : KC / 2;
    uint32_t w[W];
    __device__ __forceinline__ void load(const QT *row, bool valid) {  // row: the head's KC channels of this thread
#pragma unroll
        for (int i = 0; i < W; ++i) w[i] = valid ? __ldg(reinterpret_cast<const uint32_t *>(row) + i) : 0u;
    }
    // channels 2j and 2j + 1 of the thread's run
    __device__ __forceinline__ void pair(int j, float &a, float &b) const {
        if constexpr (sizeof(QT) == 4) {
            a = __uint_as_float(w[2 * j]);
            b = __uint_as_float(w[2 * j + 1]);
        } else {
            unpack2<QT>(w[j], a, b);
        }
    }
};

// QT: type of q_dec; CT: type of the system-token cache and of the output; D: head dim; BITS: width of a code
template <typename QT, typename CT, int D, int BITS>
__global__ void __launch_bounds__(kAtThreads, 1) attend_kernel(const AttendParams p) {
    constexpr int KS = D / 16;  // k-steps of the score product (16 channels each)
    constexpr int KC = D / 4;   // channels of a token row one thread owns in the score product
    constexpr int MT = D / 16;  // m-tiles of the value product (16 channels each)
    constexpr int VC = D / 8;   // channels one thread owns in the value product
    constexpr int KB = KC * BITS / 8, VB = VC * BITS / 8;  // bytes of packed codes behind them
    constexpr int MH = MT < 8 ? MT : 8;  // m-tiles of the value product done in one pass over the weights
    constexpr int OP = at_opitch(D), OF = at_ofloats(D);
    using BF = __nv_bfloat16;
    static_assert(kAtHeads == 8 && kAtUnitTokens == 64 && kAtSysTokens == 16, "fragment mapping");
    extern __shared__ __align__(128) unsigned char smem[];
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kAtOffAbort);
    float *stat = reinterpret_cast<float *>(smem + kAtOffStat);
    float *blk = reinterpret_cast<float *>(smem + kAtOffBlk);
    float *ob = reinterpret_cast<float *>(smem + kAtOffOb);
    unsigned char *ring = smem + at_off_ring(D);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;  // fragment coordinates of the thread
    const int h = blockIdx.y, li = blockIdx.z;
    const int G = p.g.G, H = p.g.H, md = p.g.meta_dtype, S = p.n_stages;
    const uint32_t C = cluster_size(), r = cluster_rank();
    float *wt = reinterpret_cast<float *>(smem + kAtOffWt) + warp * (kAtHeads * kAtWPitch);
    unsigned char *my_ring = ring + (size_t)warp * S * p.stage_bytes;
    const uint32_t bar0 = smem_u32(smem + kAtOffBars) + 8u * (warp * kAtMaxStages);

    if (lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(bar0 + 8 * s, 1);
        if (warp == 0) {
            abort_flag[0] = 0;  // raised by the first warp whose wait ran out
            abort_flag[1] = 0;  // never raised: lets a warp wait out its own copies regardless
        }
        mbar_init_fence();
    }
    __syncthreads();

    // ---- the units of this warp: u = u_first + i * u_step, i < n_mine
    const int u_step = (int)C * kAtWarps, u_first = (int)r + (int)C * warp;
    const int n_mine = u_first < p.n_units ? (p.n_units - u_first + u_step - 1) / u_step : 0;
    const int code_block = G * p.g.row_bytes;              // bytes of the K (or V) codes of a unit
    const int meta_row = D * (md == STOM_FP32 ? 4 : 2);    // bytes of one metadata row
    const CT *ksys = reinterpret_cast<const CT *>(p.ksys) + (int64_t)li * p.s_sl + (int64_t)h * p.s_sh;
    const CT *vsys = reinterpret_cast<const CT *>(p.vsys) + (int64_t)li * p.s_sl + (int64_t)h * p.s_sh;
    const int32_t *idx_row = p.idx + (p.per_head ? ((int64_t)li * H + h) * p.k : (int64_t)li * p.k);

    uint32_t phase_bits = 0;   // bit s: parity the next wait on stage s asks for
    uint32_t stage_info = 0;   // byte s: token count of the unit in stage s (0: nothing was posted), bit 7: system tokens
    bool dead = false;         // a wait ran out: the warp posts nothing more and its result is void

    // Group index of unit number i of this warp (lane-parallel: 32 units per load)
    auto load_tg_batch = [&](int i0) -> int32_t {
        const int u = u_first + (i0 + lane) * u_step;
        if (i0 + lane < n_mine && u >= p.n_sys_units) return __ldg(idx_row + (u - p.n_sys_units));
        return -1;
    };
    // Posts the copies of unit number i into stage i % S.  tg: the unit's group index (groups only).  Warp-collective.
    auto post_unit = [&](int i, int32_t tg) {
        const int s = i % S;
        const int u = u_first + i * u_step;
        unsigned char *st = my_ring + (size_t)s * p.stage_bytes;
        const uint32_t bar = bar0 + 8 * s, dst = smem_u32(st);
        uint32_t info = 0;
        if (u < p.n_sys_units) {
            const int tok0 = u * kAtSysTokens, n_tok = min(kAtSysTokens, p.sys_len - tok0);
            const uint32_t row = D * (uint32_t)sizeof(CT);
            info = (uint32_t)n_tok | 0x80u;
            if (lane == 0) mbar_expect_tx(bar, 2u * n_tok * row);
            __syncwarp();
            if (p.s_st == D) {  // adjacent rows: one copy each for K and V
                if (lane == 0) bulk_load(dst, ksys + (int64_t)tok0 * D, n_tok * row, bar);
                if (lane == 1) bulk_load(dst + kAtSysTokens * row, vsys + (int64_t)tok0 * D, n_tok * row, bar);
            } else if (lane < 2 * kAtSysTokens) {
                const int rr = lane & (kAtSysTokens - 1);
                if (rr < n_tok) {
                    const CT *src = (lane < kAtSysTokens ? ksys : vsys) + (int64_t)(tok0 + rr) * p.s_st;
                    bulk_load(dst + (lane < kAtSysTokens ? 0u : kAtSysTokens * row) + rr * row, src, row, bar);
                }
            }
        } else if (tg >= 0 && tg < p.n_groups) {
            const int64_t slot = bank_slot(p.g, p.layer_begin + li, tg, h);
            info = (uint32_t)G;
            if (lane == 0) mbar_expect_tx(bar, 2u * code_block + 4u * meta_row);
            __syncwarp();
            const int esz = md == STOM_FP32 ? 4 : 2;
            if (lane == 0) bulk_load(dst, p.codes_k + slot * code_block, code_block, bar);
            if (lane == 1) bulk_load(dst + code_block, p.codes_v + slot * code_block, code_block, bar);
            if (lane >= 2 && lane < 6) {
                const void *base = lane == 2 ? p.scale_k : (lane == 3 ? p.zero_k : (lane == 4 ? p.scale_v : p.zero_v));
                bulk_load(dst + 2 * code_block + (lane - 2) * meta_row,
                          static_cast<const unsigned char *>(base) + slot * D * esz, meta_row, bar);
            }
        } else if (tg != -1 && p.flags && lane == 0) {
            atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
        }
        stage_info = (stage_info & ~(0xFFu << (8 * s))) | (info << (8 * s));
    };

    for (int h0 = 0; h0 < p.rep; h0 += kAtHeads) {
        const int nh = min(kAtHeads, p.rep - h0);
        // ---- start the first units on their way, then fetch the query rows behind them
        int32_t tg_batch = load_tg_batch(0);
        if (!dead)
            for (int i = 0; i < S && i < n_mine; ++i) post_unit(i, __shfl_sync(0xffffffffu, tg_batch, i));
        QRegs<QT, KC> qr;  // query head g of the chunk, channels KC*t .. KC*t + KC - 1
        qr.load(reinterpret_cast<const QT *>(p.q) + (int64_t)li * p.q_sl + (int64_t)(h * p.rep + h0 + g) * p.q_sh + KC * t, g < nh);

        float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.0f, l_b = 0.0f;  // running max / sum of query heads 2t, 2t + 1
        float O[MT][4];  // running output: channels VC*g + 2*mm (+1) x query heads 2t, 2t + 1
#pragma unroll
        for (int mm = 0; mm < MT; ++mm)
#pragma unroll
            for (int i = 0; i < 4; ++i) O[mm][i] = 0.0f;

        for (int i = 0; i < n_mine && !dead; ++i) {
            const int s = i % S;
            const uint32_t info = (stage_info >> (8 * s)) & 0xFFu;
            const int n_tok = (int)(info & 0x7Fu);
            const bool is_sys = (info & 0x80u) != 0;
            const unsigned char *st = my_ring + (size_t)s * p.stage_bytes;
            if (n_tok > 0) {
                const bool ok = mbar_wait_bounded(bar0 + 8 * s, (phase_bits >> s) & 1u, abort_flag, kAtWaitLimitNs);
                if (!__all_sync(0xffffffffu, ok)) {
                    if (lane == 0) {
                        if (p.flags) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
                        *abort_flag = 1;
                    }
                    dead = true;
                    break;
                }
                phase_bits ^= 1u << s;
                stage_info &= ~(0xFFu << (8 * s));  // consumed: nothing of this stage is in flight any more

                // ---- phase 1: scores.  Contraction slot (kk; 2t, 2t+1, 2t+8, 2t+9) of the matrix product stands for
                //      channels KC*t + 4*kk + (0, 1, 2, 3); column g is query head g.
                const int n_mt = (n_tok + 15) >> 4;
                float sc[kAtUnitTokens / 16][4];
                {
                    uint32_t qb[KS][2], ql[KS][2];  // the thread's column of the right-hand operand, high and low parts
                    float bias = 0.0f;              // what the raw-code product leaves out, for query head g
                    if (!is_sys) {
                        const unsigned char *sk = st + 2 * code_block, *mk = sk + meta_row;
#pragma unroll
                        for (int c8 = 0; c8 < KC / 8; ++c8) {
                            float s8[8], m8[8];
                            lds_meta8(sk, KC * t + c8 * 8, md, s8);
                            lds_meta8(mk, KC * t + c8 * 8, md, m8);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {  // 2 channels each
                                const int c = c8 * 8 + 2 * j;
                                float q0, q1;
                                qr.pair(c / 2, q0, q1);
                                uint32_t whi, wlo;
                                float r0, r1;  // the two products as the tensor core sees them
                                split2<BF>(q0 * s8[2 * j], q1 * s8[2 * j + 1], whi, wlo, r0, r1);
                                bias = fmaf(q0, m8[2 * j], bias);
                                bias = fmaf(q1, m8[2 * j + 1], bias);
                                bias = fmaf(-128.0f, r0 + r1, bias);
                                qb[c / 4][(c / 2) & 1] = whi;
                                ql[c / 4][(c / 2) & 1] = wlo;
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < KC / 2; ++j) {
                            float q0, q1, r0, r1;
                            qr.pair(j, q0, q1);
                            split2<CT>(q0, q1, qb[j / 2][j & 1], ql[j / 2][j & 1], r0, r1);
                        }
                    }
                    bias += __shfl_xor_sync(0xffffffffu, bias, 1);
                    bias += __shfl_xor_sync(0xffffffffu, bias, 2);
                    const float bias_a = __shfl_sync(0xffffffffu, bias, (2 * t) << 2);       // of query head 2t
                    const float bias_b = __shfl_sync(0xffffffffu, bias, (2 * t + 1) << 2);   // of query head 2t + 1
                    // Two m-tiles at a time, and the high and low part of the right-hand operand into accumulators of
                    // their own: four independent chains of dependent products instead of one.
#pragma unroll
                    for (int mp = 0; mp < kAtUnitTokens / 32; ++mp) {
                        float ch[2][4], cl[2][4];
#pragma unroll
                        for (int u = 0; u < 2; ++u)
#pragma unroll
                            for (int e = 0; e < 4; ++e) ch[u][e] = cl[u][e] = 0.0f;
                        if (2 * mp < n_mt) {  // warp-uniform
                            if (!is_sys) {
                                uint32_t w[2][2][(KB + 3) / 4];  // [m-tile of the pair][row g / row g + 8]: the thread's KC codes
#pragma unroll
                                for (int u = 0; u < 2; ++u)
#pragma unroll
                                    for (int v = 0; v < 2; ++v) {
                                        const int row = (2 * mp + u) * 16 + g + 8 * v;
                                        lds_code_bytes<KB>(st + row * p.g.row_bytes + t * KB, row < n_tok, w[u][v]);
                                    }
#pragma unroll
                                for (int kk = 0; kk < KS; ++kk) {
                                    // codes 4kk, 4kk+1 of the thread's run share a byte, and so do 4kk+2, 4kk+3
                                    const int ca = 4 * kk, cb = 4 * kk + 2;
                                    const int wa = code_word_of<BITS>(ca), ba = code_byte_of<BITS>(ca), fa = code_field_of<BITS>(ca);
                                    const int wb = code_word_of<BITS>(cb), bb = code_byte_of<BITS>(cb), fb = code_field_of<BITS>(cb);
#pragma unroll
                                    for (int u = 0; u < 2; ++u) {
                                        const uint32_t a0 = code_pair_bf16(code_view<BITS>(w[u][0][wa], fa), code_view<BITS>(w[u][0][wa], fa + 1), ba);
                                        const uint32_t a1 = code_pair_bf16(code_view<BITS>(w[u][1][wa], fa), code_view<BITS>(w[u][1][wa], fa + 1), ba);
                                        const uint32_t a2 = code_pair_bf16(code_view<BITS>(w[u][0][wb], fb), code_view<BITS>(w[u][0][wb], fb + 1), bb);
                                        const uint32_t a3 = code_pair_bf16(code_view<BITS>(w[u][1][wb], fb), code_view<BITS>(w[u][1][wb], fb + 1), bb);
                                        mma_16816<BF>(ch[u], a0, a1, a2, a3, qb[kk][0], qb[kk][1]);
                                        mma_16816<BF>(cl[u], a0, a1, a2, a3, ql[kk][0], ql[kk][1]);
                                    }
                                }
                            } else if (mp == 0) {  // a system-token unit is one m-tile
                                uint32_t w0[KC / 2], w1[KC / 2];  // the thread's KC channels of the two token rows, 16-bit pairs
                                lds_words_or_zero<KC / 2>(st + (g * D + KC * t) * (int)sizeof(CT), g < n_tok, w0);
                                lds_words_or_zero<KC / 2>(st + ((g + 8) * D + KC * t) * (int)sizeof(CT), g + 8 < n_tok, w1);
#pragma unroll
                                for (int kk = 0; kk < KS; ++kk) {
                                    mma_16816<CT>(ch[0], w0[2 * kk], w1[2 * kk], w0[2 * kk + 1], w1[2 * kk + 1], qb[kk][0], qb[kk][1]);
                                    mma_16816<CT>(cl[0], w0[2 * kk], w1[2 * kk], w0[2 * kk + 1], w1[2 * kk + 1], ql[kk][0], ql[kk][1]);
                                }
                            }
                        }
                        // base-2 scores; token slots without a token never win the maximum and weigh nothing
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int mt = 2 * mp + u, r0 = mt * 16 + g, r1 = r0 + 8;
                            sc[mt][0] = r0 < n_tok ? (ch[u][0] + cl[u][0] + bias_a) * p.scale_log2e : -INFINITY;
                            sc[mt][1] = r0 < n_tok ? (ch[u][1] + cl[u][1] + bias_b) * p.scale_log2e : -INFINITY;
                            sc[mt][2] = r1 < n_tok ? (ch[u][2] + cl[u][2] + bias_a) * p.scale_log2e : -INFINITY;
                            sc[mt][3] = r1 < n_tok ? (ch[u][3] + cl[u][3] + bias_b) * p.scale_log2e : -INFINITY;
                        }
                    }
                }

                // ---- phase 2: the warp's own online softmax.  New running maxima of query heads 2t, 2t + 1; the
                //      scores become weights in the warp's tile [head][token slot]; the running sums and outputs
                //      are rescaled.  The sum of the weights is taken in phase 3 from the ROUNDED weights the matrix
                //      product uses, so that numerator and denominator of the softmax average see the same weights.
                float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
                for (int mt = 0; mt < kAtUnitTokens / 16; ++mt) {
                    mx_a = fmaxf(mx_a, fmaxf(sc[mt][0], sc[mt][2]));
                    mx_b = fmaxf(mx_b, fmaxf(sc[mt][1], sc[mt][3]));
                }
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, o));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, o));
                }
                const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);  // finite: the unit has a token
                const float al_a = exp2f(m_a - mn_a), al_b = exp2f(m_b - mn_b);  // 0 on the first unit
                m_a = mn_a;
                m_b = mn_b;
#pragma unroll
                for (int mt = 0; mt < kAtUnitTokens / 16; ++mt) {
                    const int r0 = mt * 16 + g;
                    wt[(2 * t) * kAtWPitch + r0] = exp2f(sc[mt][0] - mn_a);
                    wt[(2 * t + 1) * kAtWPitch + r0] = exp2f(sc[mt][1] - mn_b);
                    wt[(2 * t) * kAtWPitch + r0 + 8] = exp2f(sc[mt][2] - mn_a);
                    wt[(2 * t + 1) * kAtWPitch + r0 + 8] = exp2f(sc[mt][3] - mn_b);
                }
                l_a *= al_a;
                l_b *= al_b;
#pragma unroll
                for (int mm = 0; mm < MT; ++mm) {
                    O[mm][0] *= al_a; O[mm][1] *= al_b; O[mm][2] *= al_a; O[mm][3] *= al_b;
                }
                __syncwarp();

                // ---- phase 3: weighted sum of the values.  Rows of the product are channels: rows g and g + 8 of
                //      m-tile mm stand for channels VC*g + 2*mm and VC*g + 2*mm + 1; the contraction runs over the
                //      unit's tokens (slot 2t, 2t+1, 2t+8, 2t+9 of k-step ks is token 16*ks + the same); columns are
                //      query heads.  d = 256 takes two passes of 8 m-tiles over the same weights.
                const unsigned char *vst = st + (is_sys ? kAtSysTokens * D * (int)sizeof(CT) : code_block);
#pragma unroll
                for (int m0 = 0; m0 < MT; m0 += MH) {
                    float acc[MH][4];
#pragma unroll
                    for (int mm = 0; mm < MH; ++mm)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[mm][e] = 0.0f;
                    float wsum = 0.0f;  // sum of the weights of query head g as the tensor core sees them
#pragma unroll
                    for (int ks = 0; ks < kAtUnitTokens / 16; ++ks) {
                        if (ks < n_mt) {  // warp-uniform
                            const int ta = ks * 16 + 2 * t;  // tokens ta, ta + 1, ta + 8, ta + 9
                            const float2 wlo = *reinterpret_cast<const float2 *>(&wt[g * kAtWPitch + ta]);
                            const float2 whi = *reinterpret_cast<const float2 *>(&wt[g * kAtWPitch + ta + 8]);
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
                                for (int e = 0; e < 4; ++e) {
                                    const int tok = ta + (e & 1) + 8 * (e >> 1);
                                    lds_code_bytes<VB>(vst + tok * p.g.row_bytes + g * VB, tok < n_tok, w[e]);
                                }
#pragma unroll
                                for (int mm = 0; mm < MH; ++mm) {
                                    // channels VC*g + 2*mm and the next one share a byte; rows g and g + 8 of the m-tile
                                    const int c = 2 * (m0 + mm);
                                    const int j = code_word_of<BITS>(c), b = code_byte_of<BITS>(c), f = code_field_of<BITS>(c);
                                    const uint32_t a0 = code_pair_bf16(code_view<BITS>(w[0][j], f), code_view<BITS>(w[1][j], f), b);
                                    const uint32_t a1 = code_pair_bf16(code_view<BITS>(w[0][j], f + 1), code_view<BITS>(w[1][j], f + 1), b);
                                    const uint32_t a2 = code_pair_bf16(code_view<BITS>(w[2][j], f), code_view<BITS>(w[3][j], f), b);
                                    const uint32_t a3 = code_pair_bf16(code_view<BITS>(w[2][j], f + 1), code_view<BITS>(w[3][j], f + 1), b);
                                    mma_16816<BF>(acc[mm], a0, a1, a2, a3, b0, b1);
                                    mma_16816<BF>(acc[mm], a0, a1, a2, a3, l0, l1);
                                }
                            } else if (ks == 0) {
                                uint32_t w[4][VC / 2];  // the thread's VC channels of its 4 tokens, 16-bit pairs (channel 2mm, 2mm+1)
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int tok = ta + (e & 1) + 8 * (e >> 1);
                                    lds_words_or_zero<VC / 2>(vst + (tok * D + VC * g) * (int)sizeof(CT), tok < n_tok, w[e]);
                                }
#pragma unroll
                                for (int mm = 0; mm < MH; ++mm) {
                                    const int j = m0 + mm;
                                    const uint32_t a0 = __byte_perm(w[0][j], w[1][j], 0x5410), a1 = __byte_perm(w[0][j], w[1][j], 0x7632);
                                    const uint32_t a2 = __byte_perm(w[2][j], w[3][j], 0x5410), a3 = __byte_perm(w[2][j], w[3][j], 0x7632);
                                    mma_16816<CT>(acc[mm], a0, a1, a2, a3, b0, b1);
                                    mma_16816<CT>(acc[mm], a0, a1, a2, a3, l0, l1);
                                }
                            }
                        }
                    }
                    wsum += __shfl_xor_sync(0xffffffffu, wsum, 1);
                    wsum += __shfl_xor_sync(0xffffffffu, wsum, 2);
                    const float ws_a = __shfl_sync(0xffffffffu, wsum, (2 * t) << 2), ws_b = __shfl_sync(0xffffffffu, wsum, (2 * t + 1) << 2);
                    if (m0 == 0) {
                        l_a += ws_a;
                        l_b += ws_b;
                    }
                    if (!is_sys) {
                        // acc holds sum_t w_t (128 + code): apply the group's scale and offset, channel by channel
                        const unsigned char *sv = st + 2 * code_block + 2 * meta_row, *mv = sv + meta_row;
#pragma unroll
                        for (int c8 = 0; c8 < 2 * MH / 8; ++c8) {
                            float s8[8], m8[8];
                            lds_meta8(sv, VC * g + 2 * m0 + c8 * 8, md, s8);
                            lds_meta8(mv, VC * g + 2 * m0 + c8 * 8, md, m8);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int mm = c8 * 4 + j;
                                O[m0 + mm][0] += fmaf(s8[2 * j], fmaf(-128.0f, ws_a, acc[mm][0]), m8[2 * j] * ws_a);
                                O[m0 + mm][1] += fmaf(s8[2 * j], fmaf(-128.0f, ws_b, acc[mm][1]), m8[2 * j] * ws_b);
                                O[m0 + mm][2] += fmaf(s8[2 * j + 1], fmaf(-128.0f, ws_a, acc[mm][2]), m8[2 * j + 1] * ws_a);
                                O[m0 + mm][3] += fmaf(s8[2 * j + 1], fmaf(-128.0f, ws_b, acc[mm][3]), m8[2 * j + 1] * ws_b);
                            }
                        }
                    } else {
#pragma unroll
                        for (int mm = 0; mm < MH; ++mm)
#pragma unroll
                            for (int e = 0; e < 4; ++e) O[m0 + mm][e] += acc[mm][e];
                    }
                }
                __syncwarp();  // every lane is done with the stage and with the weight tile
            }
            // ---- the stage is free: post the unit that comes S units later
            const int in = i + S;
            if (in < n_mine) {
                if ((in & 31) == 0) tg_batch = load_tg_batch(in);
                post_unit(in, __shfl_sync(0xffffffffu, tg_batch, in & 31));
            }
        }

        // ---- merge the warps of the block.  Each warp rescales its output to the block's maximum and parks it in its
        //      own first stage, laid out [channel slab g][channel][head] with padded slabs so that neither these
        //      stores nor the sums below collide on shared-memory banks.
        if (dead) {
            m_a = m_b = -INFINITY;
            l_a = l_b = 0.0f;
        }
        if (g == 0) {
            stat[warp * 16 + 2 * t] = m_a;
            stat[warp * 16 + 2 * t + 1] = m_b;
            stat[warp * 16 + 8 + 2 * t] = l_a;
            stat[warp * 16 + 8 + 2 * t + 1] = l_b;
        }
        // nothing of this warp may still be landing in the stage that now takes its result (only after a wait ran out)
        for (int s = 0; s < S; ++s) {
            if ((stage_info >> (8 * s)) & 0x7Fu) {
                mbar_wait_bounded(bar0 + 8 * s, (phase_bits >> s) & 1u, abort_flag + 1, kAtWaitLimitNs);
                phase_bits ^= 1u << s;
                stage_info &= ~(0xFFu << (8 * s));
            }
        }
        __syncthreads();
        {
            float M_a = -INFINITY, M_b = -INFINITY;
#pragma unroll
            for (int w = 0; w < kAtWarps; ++w) {
                M_a = fmaxf(M_a, stat[w * 16 + 2 * t]);
                M_b = fmaxf(M_b, stat[w * 16 + 2 * t + 1]);
            }
            const float f_a = m_a == -INFINITY ? 0.0f : exp2f(m_a - M_a), f_b = m_b == -INFINITY ? 0.0f : exp2f(m_b - M_b);
            float *mine = reinterpret_cast<float *>(my_ring) + g * OP + 2 * t;
#pragma unroll
            for (int mm = 0; mm < MT; ++mm) {
                *reinterpret_cast<float2 *>(mine + (2 * mm) * 8) = make_float2(O[mm][0] * f_a, O[mm][1] * f_b);
                *reinterpret_cast<float2 *>(mine + (2 * mm + 1) * 8) = make_float2(O[mm][2] * f_a, O[mm][3] * f_b);
            }
        }
        __syncthreads();
        for (int e = tid; e < OF; e += kAtThreads) {
            float a = 0.0f;
#pragma unroll
            for (int w = 0; w < kAtWarps; ++w)
                a += reinterpret_cast<const float *>(ring + (size_t)w * S * p.stage_bytes)[e];
            ob[e] = a;
        }
        if (tid < kAtHeads) {
            float M = -INFINITY, L = 0.0f;
#pragma unroll
            for (int w = 0; w < kAtWarps; ++w) M = fmaxf(M, stat[w * 16 + tid]);
#pragma unroll
            for (int w = 0; w < kAtWarps; ++w) {
                const float mw = stat[w * 16 + tid];
                if (mw != -INFINITY) L = fmaf(stat[w * 16 + 8 + tid], exp2f(mw - M), L);
            }
            blk[tid] = M;
            blk[8 + tid] = L;
        }

        // ---- merge the blocks of the cluster: rank r finishes its share of the (channel, head) pairs
        if (C > 1) cluster_sync(); else __syncthreads();
        {
            const int per = (OF + (int)C - 1) / (int)C;
            const int e_end = min(per * ((int)r + 1), OF);
            for (int e = per * (int)r + tid; e < e_end; e += kAtThreads) {
                const int slab = e / OP, rem = e - slab * OP;
                const int hh = rem & 7, cl = rem >> 3;
                if (cl >= VC || hh >= nh) continue;  // padding, or a head beyond the GQA block
                float num = 0.0f, den = 0.0f;
                if (C > 1) {
                    // every block's (max, sum, partial) of this pair is asked for before any of them is used
                    float Mb[8], Lb[8], Ov[8];
#pragma unroll
                    for (uint32_t b = 0; b < 8; ++b) {
                        Mb[b] = -INFINITY;
                        Lb[b] = Ov[b] = 0.0f;
                        if (b < C) {
                            Mb[b] = ld_cluster_f(blk + hh, b);
                            Lb[b] = ld_cluster_f(blk + 8 + hh, b);
                            Ov[b] = ld_cluster_f(ob + e, b);
                        }
                    }
                    float M = -INFINITY;
#pragma unroll
                    for (int b = 0; b < 8; ++b) M = fmaxf(M, Mb[b]);
#pragma unroll
                    for (int b = 0; b < 8; ++b) {
                        const float f = Mb[b] == -INFINITY ? 0.0f : exp2f(Mb[b] - M);
                        num = fmaf(Ov[b], f, num);
                        den = fmaf(Lb[b], f, den);
                    }
                } else {
                    num = ob[e];
                    den = blk[8 + hh];
                }
                CT *out = reinterpret_cast<CT *>(p.out) + (int64_t)li * p.o_sl + (int64_t)(h * p.rep + h0 + hh) * p.o_sh;
                out[VC * slab + cl] = (CT)(den > 0.0f ? num / den : 0.0f);
            }
        }
        // nobody leaves, or reuses its buffers for the next chunk of heads, while a neighbour still reads from them
        if (C > 1) cluster_sync(); else __syncthreads();
    }
}

static int attend_units(const stom_oqm_config *cfg, int32_t k, int32_t sys_len, int *n_sys_units) {
    *n_sys_units = (sys_len + kAtSysTokens - 1) / kAtSysTokens;
    return *n_sys_units + k;
}

// bytes of one ring stage: a group's K and V codes and its four metadata rows, or 16 system tokens of K and of V
static int attend_stage_bytes(const stom_oqm_config *cfg) {
    const int group = 2 * cfg->group_tokens * (cfg->head_dim * cfg->bits / 8) + 4 * cfg->head_dim * elem_bytes(cfg->meta_dtype);
    const int sys = 2 * kAtSysTokens * cfg->head_dim * 2;
    const int b = group > sys ? group : sys;
    return (b + 127) / 128 * 128;
}

template <typename KernelT>
static int32_t launch_attend_kernel(KernelT kernel, const AttendParams &p, int D, int units, int pairs_h, int layers,
                                    cudaStream_t s) {
    int dev = 0, sms = 0, smem_max = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    AttendParams q = p;
    const int fixed = at_off_ring(D);
    q.n_stages = fixed + kAtWarps * 2 * q.stage_bytes <= smem_max ? 2 : 1;
    const size_t smem = (size_t)fixed + (size_t)kAtWarps * q.n_stages * q.stage_bytes;
    if ((int64_t)smem > smem_max) return STOM_ERR_SHAPE;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    // Blocks per (layer, kv head): as many as keep every block busy for the same number of rounds of units without
    // sending more blocks to a multiprocessor than the others get; more blocks on a tie (fewer bytes per block).
    const int64_t pairs = (int64_t)pairs_h * layers;
    int best_c = 1;
    int64_t best_cost = INT64_MAX;
    for (int c = 1; c <= 8; ++c) {
        if (c > 1 && (c - 1) * kAtWarps >= units) break;  // the last block would have nothing to do
        const int64_t per_sm = (pairs * c + sms - 1) / sms;
        const int64_t rounds = (units + c * kAtWarps - 1) / (c * kAtWarps);
        const int64_t cost = per_sm * rounds;
        if (cost <= best_cost) {
            best_cost = cost;
            best_c = c;
        }
    }
    cudaLaunchConfig_t lc = {};
    lc.blockDim = dim3(kAtThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    for (int c = best_c;; --c) {
        lc.gridDim = dim3((unsigned)c, (unsigned)pairs_h, (unsigned)layers);
        at[0].val.clusterDim.x = (unsigned)c;
        int resident = 0;
        if (c == 1 || (cudaOccupancyMaxActiveClusters(&resident, kernel, &lc) == cudaSuccess && resident >= 1)) break;
        (void)cudaGetLastError();
    }
    e = cudaLaunchKernelEx(&lc, kernel, q);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    return finish_launch();
}

template <typename QT, typename CT>
static int32_t launch_attend(const AttendParams &p, int units, int layers, cudaStream_t s) {
    const bool b4 = p.g.row_bytes * 2 == p.g.d;  // 4-bit codes: d/2 bytes per row
    const int H = p.g.H;
    switch (p.g.d) {
    case 64:
        return b4 ? launch_attend_kernel(attend_kernel<QT, CT, 64, 4>, p, 64, units, H, layers, s)
                  : launch_attend_kernel(attend_kernel<QT, CT, 64, 2>, p, 64, units, H, layers, s);
    case 128:
        return b4 ? launch_attend_kernel(attend_kernel<QT, CT, 128, 4>, p, 128, units, H, layers, s)
                  : launch_attend_kernel(attend_kernel<QT, CT, 128, 2>, p, 128, units, H, layers, s);
    case 256:
        return b4 ? launch_attend_kernel(attend_kernel<QT, CT, 256, 4>, p, 256, units, H, layers, s)
                  : launch_attend_kernel(attend_kernel<QT, CT, 256, 2>, p, 256, units, H, layers, s);
    default: return STOM_ERR_SHAPE;
    }
}

}  // namespace stom

using namespace stom;

extern "C" int64_t stom_oqm_attend_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count, int32_t k,
                                                   int32_t sys_len) {
    if (check_config(cfg) || layer_count < 0 || k < 0 || sys_len < 0) return STOM_ERR_INVALID_ARG;
    return 256;  // the call keeps nothing in global memory; a token size so that callers written for a workspace keep working
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
    (void)workspace;
    (void)workspace_bytes;
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
    // a thread reads its query channels as 32-bit words
    if ((q_stride_layer * elem_bytes(cfg->kv_dtype)) % 4 || (q_stride_head * elem_bytes(cfg->kv_dtype)) % 4)
        return STOM_ERR_ALIGNMENT;
    if (sys_len > 0 && (!aligned16(k_sys) || !aligned16(v_sys) || !stride_ok(sys_stride_layer, cache_dtype) ||
                        !stride_ok(sys_stride_head, cache_dtype) || !stride_ok(sys_stride_token, cache_dtype)))
        return STOM_ERR_ALIGNMENT;
    if (layer_count == 0) return STOM_OK;

    AttendParams p;
    p.idx = idx;
    p.codes_k = store->codes_k; p.codes_v = store->codes_v;
    p.scale_k = store->scale_k; p.zero_k = store->zero_k; p.scale_v = store->scale_v; p.zero_v = store->zero_v;
    p.q = q_dec; p.q_sl = q_stride_layer; p.q_sh = q_stride_head;
    p.ksys = k_sys; p.vsys = v_sys; p.s_sl = sys_stride_layer; p.s_sh = sys_stride_head; p.s_st = sys_stride_token;
    p.out = out; p.o_sl = out_stride_layer; p.o_sh = out_stride_head;
    p.g = bank_geom(cfg);
    p.layer_begin = layer_begin; p.k = k; p.n_groups = n_groups;
    p.per_head = cfg->score_mode == STOM_SCORE_PER_HEAD;
    p.rep = cfg->n_q_heads / cfg->n_kv_heads;
    p.sys_len = sys_len;
    p.n_units = attend_units(cfg, k, sys_len, &p.n_sys_units);
    p.stage_bytes = attend_stage_bytes(cfg);
    p.n_stages = 1;
    p.scale_log2e = softmax_scale * 1.4426950408889634f;
    p.flags = dev_flags;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (layer_count > 65535 || cfg->n_kv_heads > 65535) return STOM_ERR_SHAPE;
    const bool bf = cache_dtype == STOM_BF16;
    switch (cfg->kv_dtype) {
    case STOM_BF16:
        return bf ? launch_attend<__nv_bfloat16, __nv_bfloat16>(p, p.n_units, layer_count, s)
                  : launch_attend<__nv_bfloat16, __half>(p, p.n_units, layer_count, s);
    case STOM_FP16:
        return bf ? launch_attend<__half, __nv_bfloat16>(p, p.n_units, layer_count, s)
                  : launch_attend<__half, __half>(p, p.n_units, layer_count, s);
    default:
        return bf ? launch_attend<float, __nv_bfloat16>(p, p.n_units, layer_count, s)
                  : launch_attend<float, __half>(p, p.n_units, layer_count, s);
    }
}
