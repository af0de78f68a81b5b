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
//   team     the warps that work on one unit together.  The kernel comes in
//            two shapes.  Four warps per team, warp j on tokens 16j .. 16j+15
//            of the group: the shortest path through one unit, for calls that
//            are latency (a decoder calling layer by layer).  Two warps per
//            team, each walking two 16-token tiles: fewer instructions per
//            unit (the team's shared preparation is paid once per two tiles)
//            and eight teams with a ring of two stages each in one block, for
//            calls with many units per multiprocessor (all layers at once):
//            the next unit is on its way while a team works on this one.
//            The right-hand operand of
//            the score product (q * s of the group, as a high and a low
//            16-bit part) is the same for all tokens: the team prepares it
//            once per unit, each warp a share, and passes it through shared
//            memory with one barrier of the team per unit; that barrier also
//            tells the team that the unit before is consumed, so its ring
//            stage is posted again.  Per unit a warp computes the scores of
//            its tokens (a tensor-core product over the raw codes), its own
//            online softmax, and its share of the weighted sum of V (again a
//            tensor-core product over raw codes); it keeps a running (max,
//            sum, output) for the 8 query heads it handles
//   merge    the warps of a block combine through shared memory, the blocks
//            of the cluster through distributed shared memory (one hardware
//            cluster barrier on each side); rank r writes its share of the
//            output rows.  No workspace, no tickets, nobody spins on memory.
#include <mutex>

#include "stom_async.cuh"
#include "stom_internal.cuh"

namespace stom {

constexpr int kAtMaxWarps = 16;
constexpr int kAtMaxThreads = kAtMaxWarps * 32;
constexpr int kAtSysTokens = 16;   // tokens of a system-token unit (one 16-token tile)
constexpr int kAtHeads = 8;        // query heads handled together
constexpr int kAtMaxStages = 3;
constexpr int kAtMaxCluster = 16;
constexpr unsigned long long kAtWaitLimitNs = 2000000000ull;  // a copy that has not landed after 2 s ends the block

// Shared-memory layout of a block of `teams` teams of 4 / MPW warps (byte offsets into dynamic shared memory)
struct AtLayout {
    int off_abort, off_stat, off_blk, off_wt, off_ob, off_xchg, off_ring, ring_bytes, total;
};
__host__ __device__ constexpr int at_wpitch(int MPW) { return 16 * MPW + 4; }  // floats per head row of a warp's weight tile
__host__ __device__ constexpr int at_xchg_bytes(int D, int MPW) { return (D / 16) * 32 * 16 + (4 / MPW) * 32 * 4; }  // operand parts + bias parts
__host__ __device__ inline AtLayout at_layout(int D, int MPW, int teams, int stages, int stage_bytes) {
    const int warps = teams * (4 / MPW);
    AtLayout l;
    l.off_abort = kAtMaxWarps * kAtMaxStages * 8;                   // after the mbarriers [teams][kAtMaxStages]
    l.off_stat = l.off_abort + 128;                                 // [warps][16]: max[8], sum[8] of each warp
    l.off_blk = l.off_stat + warps * 64;                            // max[8], sum[8] of the block
    l.off_wt = l.off_blk + 64;                                      // [warps][8][wpitch] weights
    l.off_ob = l.off_wt + warps * kAtHeads * at_wpitch(MPW) * 4;    // the block's partial output [8 * D]
    l.off_xchg = l.off_ob + 8 * D * 4;                              // [teams][2 or 1] exchange buffers
    l.off_ring = (l.off_xchg + teams * (MPW == 4 ? 1 : 2) * at_xchg_bytes(D, MPW) + 127) / 128 * 128;
    const int park = warps * 8 * D * 4;                             // the ring also takes the warps' results at the end
    l.ring_bytes = teams * stages * stage_bytes > park ? teams * stages * stage_bytes : park;
    l.total = l.off_ring + l.ring_bytes;
    return l;
}

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
    int32_t stage_bytes, n_stages, teams;
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
// and the matrix operand is the raw code.  A code becomes a bfloat16 without arithmetic: with the 4 code bits moved
// to bits 3..6 of a byte, 0x4180 | byte is the number 16 + code, exactly (2-bit codes: 0x4080 | code << 5 is 4 + code);
// the 16 is taken out again through the same sums.  The contraction index of a matrix product may be permuted freely
// as long as both operands use the same permutation, and so may the output columns: a thread therefore owns
// CONTIGUOUS code bytes (for the scores: d/4 adjacent channels of a token row; for the values: d/8 adjacent channels
// of four tokens), which it loads with one vector load and slices with byte permutes.
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

// 2^x for x <= 0 (and a little above); -inf gives 0
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// NW 32-bit words from shared memory at p (aligned to min(16, 4 * NW) bytes)
template <int NW>
__device__ __forceinline__ void lds_words(const unsigned char *p, uint32_t (&w)[NW]) {
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
template <int NW>
__device__ __forceinline__ void lds_words_or_zero(const unsigned char *p, bool valid, uint32_t (&w)[NW]) {
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = 0u;
    if (valid) lds_words<NW>(p, w);
}
// NB bytes of packed codes from shared memory at p (aligned to min(16, NB) bytes) as 32-bit words
template <int NB>
__device__ __forceinline__ void lds_code_bytes(const unsigned char *p, uint32_t (&w)[(NB + 3) / 4]) {
    if constexpr (NB == 2) w[0] = (uint32_t)*reinterpret_cast<const uint16_t *>(p);
    else lds_words<NB / 4>(p, w);
}

// How a code of BITS bits sits in a bfloat16: the byte (code << SH) | 0x80 under the high byte HI is the number OFF + code
template <int BITS> struct CodeFmt;
template <> struct CodeFmt<4> { static constexpr int SH = 3; static constexpr uint32_t MASK = 0x78787878u, HI = 0x41u; static constexpr float OFF = 16.0f; };
template <> struct CodeFmt<2> { static constexpr int SH = 5; static constexpr uint32_t MASK = 0x60606060u, HI = 0x40u; static constexpr float OFF = 4.0f; };

// Field f of every byte of a word of packed codes (a byte holds 8/BITS codes, lowest channel in the lowest bits):
// byte b of the result is (code of channel (8/BITS) * b + f of the word) << SH, alone in its byte; with OR80 the
// byte's top bit is set too (the low byte of the bfloat16 is then complete).
template <int BITS, bool OR80>
__device__ __forceinline__ uint32_t code_view(uint32_t w, int f) {
    const int sh = CodeFmt<BITS>::SH - BITS * f;
    const uint32_t x = sh >= 0 ? (w << sh) : (w >> -sh);
    return OR80 ? ((x & CodeFmt<BITS>::MASK) | 0x80808080u) : (x & CodeFmt<BITS>::MASK);
}
// Where code i of a run of packed codes sits: word, byte of the word, field of the byte.
template <int BITS> __device__ __forceinline__ constexpr int code_word_of(int i) { return i / (32 / BITS); }
template <int BITS> __device__ __forceinline__ constexpr int code_byte_of(int i) { return (i % (32 / BITS)) / (8 / BITS); }
template <int BITS> __device__ __forceinline__ constexpr int code_field_of(int i) { return i % (8 / BITS); }

// Byte `b` of x and byte `b` of y (plain views) as the bfloat16 pair (OFF + code of x, OFF + code of y): the permute
// puts the two bytes into the low byte of each half and fills the other two with the sign of a source byte (selector
// values of 8 and above), which is zero; the rest of the number is OR-ed in.
template <int BITS>
__device__ __forceinline__ uint32_t code_pair(uint32_t x, uint32_t y, int b) {
    uint32_t v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(v) : "r"(x), "r"(y), "r"(0x8480u + (uint32_t)b * 0x0101u));
    return v | (CodeFmt<BITS>::HI * 0x01000100u + 0x00800080u);
}
// Bytes `b0` and `b1` of one view taken with OR80, as the bfloat16 pair: one permute against a word of high bytes
template <int BITS>
__device__ __forceinline__ uint32_t code_pair_same(uint32_t x, int b0, int b1) {
    uint32_t v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(v) : "r"(x), "r"(CodeFmt<BITS>::HI * 0x01010101u), "r"(0x4040u + (uint32_t)b0 + ((uint32_t)b1 << 8)));
    return v;
}

// Two floats as a (high, low) pair of packed 16-bit pairs: hi = the values rounded to MT, lo = what the rounding
// left over, rounded again.  A matrix product issued once with each part carries 16 significant bits of the operand.
template <typename MT>
__device__ __forceinline__ void split2(float a, float b, uint32_t &hi, uint32_t &lo) {
    hi = pack2<MT>(a, b);
    float ha, hb;
    unpack2<MT>(hi, ha, hb);
    lo = pack2<MT>(a - ha, b - hb);
}

// Eight / four adjacent metadata values (element type by the run-time code md) from shared memory, as floats
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
__device__ __forceinline__ void lds_meta4(const unsigned char *row, int ch, int md, float (&f)[4]) {
    if (md == STOM_FP32) {
        const float4 a = *reinterpret_cast<const float4 *>(row + ch * 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
    } else {
        const uint2 v = *reinterpret_cast<const uint2 *>(row + ch * 2);
        if (md == STOM_BF16) {
            unpack2<__nv_bfloat16>(v.x, f[0], f[1]); unpack2<__nv_bfloat16>(v.y, f[2], f[3]);
        } else {
            unpack2<__half>(v.x, f[0], f[1]); unpack2<__half>(v.y, f[2], f[3]);
        }
    }
}

// barrier of the n threads of one team (hardware barrier `id`, 1 .. 15; 0 is the block's)
__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// N query channels of one head, kept in registers in the type they arrive in
template <typename QT, int N>
struct QRegs {
    static constexpr int W = sizeof(QT) == 4 ? N : N / 2;
    uint32_t w[W];
    __device__ __forceinline__ void load(const QT *at, bool valid) {
#pragma unroll
        for (int i = 0; i < W; ++i) w[i] = valid ? __ldg(reinterpret_cast<const uint32_t *>(at) + i) : 0u;
    }
    // channels 2j and 2j + 1 of the run
    __device__ __forceinline__ void pair(int j, float &a, float &b) const {
        if constexpr (sizeof(QT) == 4) {
            a = __uint_as_float(w[2 * j]);
            b = __uint_as_float(w[2 * j + 1]);
        } else {
            unpack2<QT>(w[j], a, b);
        }
    }
};

// Where element (channel slab g, channel c of the slab, query head) of a partial output sits: slabs of VC channels x 8
// heads, the channels of slab g rotated by g so that the fragment stores of a warp fall on different banks.
template <int VC>
__device__ __forceinline__ int at_oidx(int slab, int c, int head) { return slab * (VC * 8) + ((c + slab) % VC) * 8 + head; }

// QT: type of q_dec; CT: type of the system-token cache and of the output; D: head dim; BITS: width of a code;
// MPW: 16-token tiles of a unit that one warp takes (1: four warps per team; 2: two; 4: one warp per team)
template <typename QT, typename CT, int D, int BITS, int MPW>
__global__ void __launch_bounds__(kAtMaxThreads, 1) attend_kernel(const AttendParams p) {
    constexpr int TW = 4 / MPW;  // warps per team
    constexpr int KS = D / 16;   // k-steps of the score product (16 channels each)
    constexpr int KC = D / 4;    // channels of a token row one thread owns in the score product
    constexpr int MT = D / 16;   // m-tiles of the value product (16 channels each)
    constexpr int VC = D / 8;    // channels one thread owns in the value product
    constexpr int KB = KC * BITS / 8, VB = VC * BITS / 8;  // bytes of packed codes behind them
    constexpr int MH = MT < 8 ? MT : 8;  // m-tiles of the value product done in one pass over the weights
    constexpr int NPK = KS / TW;         // k-steps of the score product's right-hand operand one warp prepares
    constexpr int MP = MPW < 2 ? MPW : 2;  // token tiles whose score products run side by side
    constexpr int WP = at_wpitch(MPW);
    constexpr int XB = at_xchg_bytes(D, MPW), NXB = TW > 1 ? 2 : 1;
    constexpr bool kSameView = BITS == 4;  // score product: both codes of an operand register come from one view
    constexpr float kOff = CodeFmt<BITS>::OFF;
    using BF = __nv_bfloat16;
    static_assert(kAtHeads == 8 && kAtSysTokens == 16 && (MPW == 1 || MPW == 2 || MPW == 4), "fragment mapping");
    extern __shared__ __align__(128) unsigned char smem[];
    const AtLayout lay = at_layout(D, MPW, p.teams, p.n_stages, p.stage_bytes);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + lay.off_abort);
    float *stat = reinterpret_cast<float *>(smem + lay.off_stat);
    float *blk = reinterpret_cast<float *>(smem + lay.off_blk);
    float *ob = reinterpret_cast<float *>(smem + lay.off_ob);
    unsigned char *ring = smem + lay.off_ring;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = p.teams * TW, n_threads = n_warps * 32;
    const int team = warp / TW, wj = warp % TW;  // the warp takes token tiles wj * MPW .. wj * MPW + MPW - 1 of a unit
    const int g = lane >> 2, t = lane & 3;       // fragment coordinates of the thread
    const int h = blockIdx.y, li = blockIdx.z;
    const int G = p.g.G, H = p.g.H, md = p.g.meta_dtype, S = p.n_stages;
    const uint32_t C = cluster_size(), r = cluster_rank();
    float *wt = reinterpret_cast<float *>(smem + lay.off_wt) + warp * (kAtHeads * WP);
    unsigned char *my_ring = ring + (size_t)team * S * p.stage_bytes;
    unsigned char *xchg = smem + lay.off_xchg + team * NXB * XB;
    const uint32_t bar0 = smem_u32(smem) + 8u * (team * kAtMaxStages);
    auto team_sync = [&]() {
        if constexpr (TW == 1) __syncwarp();
        else named_sync(1 + team, 32 * TW);
    };

    // The launch may overlap the tail of the kernel ahead of it in the stream (programmatic dependent launch): what
    // follows up to the wait touches shared memory only; the kernel behind this one may be scheduled from here on
    // and does its own waiting.
    grid_launch_dependents();
    if (wj == 0 && lane == 0) {
        for (int s = 0; s < S; ++s) mbar_init(bar0 + 8 * s, 1);
        if (warp == 0) {
            abort_flag[0] = 0;  // raised by the first warp whose wait ran out
            abort_flag[1] = 0;  // never raised: lets a team wait out its own copies regardless
        }
        mbar_init_fence();
    }
    __syncthreads();

    // ---- the units of this team: u = u_first + i * u_step, i < n_mine
    const int u_step = (int)C * p.teams, u_first = (int)r * p.teams + team;
    const int n_mine = u_first < p.n_units ? (p.n_units - u_first + u_step - 1) / u_step : 0;
    const int code_block = G * p.g.row_bytes;              // bytes of the K (or V) codes of a unit
    const int meta_row = D * (md == STOM_FP32 ? 4 : 2);    // bytes of one metadata row
    const CT *ksys = reinterpret_cast<const CT *>(p.ksys) + (int64_t)li * p.s_sl + (int64_t)h * p.s_sh;
    const CT *vsys = reinterpret_cast<const CT *>(p.vsys) + (int64_t)li * p.s_sl + (int64_t)h * p.s_sh;
    const int32_t *idx_row = p.idx + (p.per_head ? ((int64_t)li * H + h) * p.k : (int64_t)li * p.k);

    uint32_t phase_bits = 0;  // bit s: parity the next wait on stage s asks for
    uint32_t stage_info = 0;  // byte s: token count of the unit posted into stage s and not yet waited for (0: none), bit 7: system tokens
    bool dead = false;        // a wait ran out: the warp computes nothing more, but keeps meeting its team's barriers

    // The six copies of a group unit, one per lane 0..5 (lane c of warp c % TW issues copy c): K codes, V codes, and
    // the four metadata rows.  A lane keeps where its array starts for this (layer, kv head), how far apart two groups
    // are in it, how many bytes a unit has of it, and where they go inside a stage.
    const unsigned char *cp_base = nullptr;
    int64_t cp_stride = 0;
    uint32_t cp_bytes = 0, cp_dst = 0;
    if (lane < 6) {
        const int esz = md == STOM_FP32 ? 4 : 2;
        const int64_t slot0 = bank_slot(p.g, p.layer_begin + li, 0, h);
        if (lane < 2) {
            cp_base = (lane == 0 ? p.codes_k : p.codes_v) + slot0 * code_block;
            cp_stride = (int64_t)H * code_block;
            cp_bytes = (uint32_t)code_block;
            cp_dst = (uint32_t)(lane * code_block);
        } else {
            const void *base = lane == 2 ? p.scale_k : (lane == 3 ? p.zero_k : (lane == 4 ? p.scale_v : p.zero_v));
            cp_base = static_cast<const unsigned char *>(base) + slot0 * D * esz;
            cp_stride = (int64_t)H * D * esz;
            cp_bytes = (uint32_t)meta_row;
            cp_dst = (uint32_t)(2 * code_block + (lane - 2) * meta_row);
        }
    }
    const bool cp_mine = lane < 6 && lane % TW == wj;
    const uint32_t group_tx = 2u * code_block + 4u * meta_row;

    // Group index of unit number i of this team (lane-parallel: 32 units per load); every warp of the team loads the
    // same words, so all of them know what was posted
    auto load_tg_batch = [&](int i0) -> int32_t {
        const int u = u_first + (i0 + lane) * u_step;
        if (i0 + lane < n_mine && u >= p.n_sys_units) return __ldg(idx_row + (u - p.n_sys_units));
        return -1;
    };
    // Posts the copies of unit number i (group index tg) into stage s: every warp of the team calls it and issues its
    // share (warp 0 also announces the byte count -- a copy that completes before the announcement only drives the
    // barrier's byte count negative for a moment, the phase cannot complete before warp 0 has arrived on it).
    auto post_unit = [&](int i, int s, int32_t tg) {
        const int u = u_first + i * u_step;
        const uint32_t bar = bar0 + 8 * s, dst = smem_u32(my_ring + (size_t)s * p.stage_bytes);
        if (u < p.n_sys_units) {
            const int tok0 = u * kAtSysTokens, n_tok = min(kAtSysTokens, p.sys_len - tok0);
            const uint32_t row = D * (uint32_t)sizeof(CT);
            stage_info |= ((uint32_t)n_tok | 0x80u) << (8 * s);
            if (wj == 0 && lane == 0) mbar_expect_tx(bar, 2u * n_tok * row);
            if (TW == 1) __syncwarp();
#pragma unroll
            for (int c = 0; c < 2; ++c) {  // copy 0: the K rows; copy 1: the V rows
                if (c % TW != wj) continue;
                const CT *src = (c == 0 ? ksys : vsys) + (int64_t)tok0 * p.s_st;
                const uint32_t to = dst + (c == 0 ? 0u : kAtSysTokens * row);
                if (p.s_st == D) {  // adjacent rows: one copy
                    if (lane == 0) bulk_load(to, src, n_tok * row, bar);
                } else if (lane < n_tok) {
                    bulk_load(to + lane * row, src + (int64_t)lane * p.s_st, row, bar);
                }
            }
        } else if (tg >= 0 && tg < p.n_groups) {
            stage_info |= (uint32_t)G << (8 * s);
            if (wj == 0 && lane == 0) mbar_expect_tx(bar, group_tx);
            if (TW == 1) __syncwarp();
            if (cp_mine) bulk_load(dst + cp_dst, cp_base + tg * cp_stride, cp_bytes, bar);
        } else if (tg != -1 && p.flags && wj == 0 && lane == 0) {
            atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
        }
    };

    // everything above is arithmetic on the arguments; from here on global memory is read
    grid_dependency_wait();  // indices, the query rows or the bank may come from the kernel just ahead in the stream
    for (int h0 = 0; h0 < p.rep; h0 += kAtHeads) {
        const int nh = min(kAtHeads, p.rep - h0);
        // ---- start the first units on their way, then fetch this warp's share of the query rows behind them
        int32_t tg_batch = load_tg_batch(0);
        if (!dead)
            for (int i = 0; i < S && i < n_mine; ++i) post_unit(i, i, __shfl_sync(0xffffffffu, tg_batch, i));
        // query head g of the chunk, channels KC*t + 4*NPK*wj .. + 4*NPK - 1: what this warp prepares for its team
        QRegs<QT, 4 * NPK> qr;
        qr.load(reinterpret_cast<const QT *>(p.q) + (int64_t)li * p.q_sl + (int64_t)(h * p.rep + h0 + g) * p.q_sh + KC * t +
                    4 * NPK * wj, g < nh);

        float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.0f, l_b = 0.0f;  // running max / sum of query heads 2t, 2t + 1
        float O[MT][4];  // running output: channels VC*g + 2*mm (+1) x query heads 2t, 2t + 1
#pragma unroll
        for (int mm = 0; mm < MT; ++mm)
#pragma unroll
            for (int i = 0; i < 4; ++i) O[mm][i] = 0.0f;

        int s = 0, s_prev = S - 1;  // stage of unit i, and of the unit before it
        for (int i = 0; i < n_mine; ++i) {
            const uint32_t info = (stage_info >> (8 * s)) & 0xFFu;
            const int n_tok = (int)(info & 0x7Fu);
            const bool is_sys = (info & 0x80u) != 0;
            const unsigned char *st = my_ring + (size_t)s * p.stage_bytes;
            unsigned char *xb = xchg + (NXB > 1 ? (i & 1) * XB : 0);
            if (n_tok > 0 && !dead) {
                bool ok = mbar_try_wait(bar0 + 8 * s, (phase_bits >> s) & 1u);
                if (!__all_sync(0xffffffffu, ok)) {  // not there yet: wait, with a limit
                    ok = mbar_wait_bounded(bar0 + 8 * s, (phase_bits >> s) & 1u, abort_flag, kAtWaitLimitNs);
                    if (!__all_sync(0xffffffffu, ok)) {
                        if (lane == 0) {
                            if (p.flags) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
                            *abort_flag = 1;
                        }
                        dead = true;
                    }
                }
                if (!dead) {
                    phase_bits ^= 1u << s;
                    stage_info &= ~(0xFFu << (8 * s));  // nothing of this stage is in flight any more
                }
            }
            if (n_tok > 0 && !dead) {
                // ---- this warp's share of the right-hand operand of the score product: q * s of the group as a high
                //      and a low 16-bit part (system tokens: q itself), and its part of what the raw-code product
                //      leaves out (sum of q * m, minus the code offset times the sum of the operand).  Operand register
                //      0 of k-step kk holds the channels of contraction slots (2t, 2t+1), register 1 those of (2t+8,
                //      2t+9): channels 4kk + (0, 2 | 1, 3) where the codes of a register come from one view of the
                //      code word, 4kk + (0, 1 | 2, 3) otherwise.
                float bias = 0.0f;
                uint32_t hi[NPK][2], lo[NPK][2];
                if (!is_sys) {
                    const unsigned char *sk = st + 2 * code_block, *mk = sk + meta_row;
                    const int c0 = KC * t + 4 * NPK * wj;
                    float qs_sum = 0.0f;
#pragma unroll
                    for (int c4 = 0; c4 < NPK; ++c4) {
                        float s4[4], m4[4], q4[4];
                        lds_meta4(sk, c0 + 4 * c4, md, s4);
                        lds_meta4(mk, c0 + 4 * c4, md, m4);
                        qr.pair(2 * c4, q4[0], q4[1]);
                        qr.pair(2 * c4 + 1, q4[2], q4[3]);
                        float x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            x[e] = q4[e] * s4[e];
                            bias = fmaf(q4[e], m4[e], bias);
                        }
                        qs_sum += (x[0] + x[1]) + (x[2] + x[3]);
                        if constexpr (kSameView) {
                            split2<BF>(x[0], x[2], hi[c4][0], lo[c4][0]);
                            split2<BF>(x[1], x[3], hi[c4][1], lo[c4][1]);
                        } else {
                            split2<BF>(x[0], x[1], hi[c4][0], lo[c4][0]);
                            split2<BF>(x[2], x[3], hi[c4][1], lo[c4][1]);
                        }
                    }
                    bias = fmaf(-kOff, qs_sum, bias);
                } else {
#pragma unroll
                    for (int c4 = 0; c4 < NPK; ++c4)
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            float q0, q1;
                            qr.pair(2 * c4 + j, q0, q1);
                            split2<CT>(q0, q1, hi[c4][j], lo[c4][j]);
                        }
                }
#pragma unroll
                for (int c4 = 0; c4 < NPK; ++c4)
                    reinterpret_cast<uint4 *>(xb)[(NPK * wj + c4) * 32 + lane] = make_uint4(hi[c4][0], hi[c4][1], lo[c4][0], lo[c4][1]);
                reinterpret_cast<float *>(xb + KS * 32 * 16)[wj * 32 + lane] = bias;
            }
            // ---- the team meets: the operand parts are out, and every warp has left the unit before this one
            team_sync();
            if (TW > 1 && i > 0 && i - 1 + S < n_mine && !dead) {  // that unit's stage takes the unit S - 1 ahead of this one
                const int in = i - 1 + S;
                const int32_t tb = (in >> 5) == (i >> 5) ? tg_batch : load_tg_batch(in & ~31);
                post_unit(in, s_prev, __shfl_sync(0xffffffffu, tb, in & 31));
            }
            const int tile0 = wj * MPW;                      // first 16-token tile of this warp
            const int n_tiles = min(MPW, (n_tok + 15 - 16 * tile0) >> 4);  // tiles of the unit that fall to this warp
            if (n_tiles > 0 && !dead) {
                // ---- phase 1: scores of this warp's tokens.  Column g of the product is query head g.
                float sc[MPW][4];
                {
                    float bias = 0.0f;
                    const float *bp = reinterpret_cast<const float *>(xb + KS * 32 * 16);
#pragma unroll
                    for (int w = 0; w < TW; ++w) bias += bp[w * 32 + lane];
                    bias += __shfl_xor_sync(0xffffffffu, bias, 1);
                    bias += __shfl_xor_sync(0xffffffffu, bias, 2);
                    const float bias_a = __shfl_sync(0xffffffffu, bias, (2 * t) << 2);       // of query head 2t
                    const float bias_b = __shfl_sync(0xffffffffu, bias, (2 * t + 1) << 2);   // of query head 2t + 1
#pragma unroll
                    for (int ip = 0; ip < MPW; ip += MP) {
                        // MP tiles side by side, and the high and low part of the right-hand operand into accumulators of
                        // their own: 2 * MP independent chains of dependent products
                        float ch[MP][4], cl[MP][4];
#pragma unroll
                        for (int u = 0; u < MP; ++u)
#pragma unroll
                            for (int e = 0; e < 4; ++e) ch[u][e] = cl[u][e] = 0.0f;
                        if (ip < n_tiles) {  // warp-uniform
                            if (!is_sys) {
                                uint32_t w[MP][2][(KB + 3) / 4];  // [tile][row g / row g + 8]: the thread's KC codes
#pragma unroll
                                for (int u = 0; u < MP; ++u)
#pragma unroll
                                    for (int v = 0; v < 2; ++v)
                                        lds_code_bytes<KB>(st + ((tile0 + ip + u) * 16 + g + 8 * v) * p.g.row_bytes + t * KB, w[u][v]);
#pragma unroll
                                for (int kk = 0; kk < KS; ++kk) {
                                    const uint4 b = reinterpret_cast<const uint4 *>(xb)[kk * 32 + lane];
                                    const int ca = 4 * kk, cb = 4 * kk + 2;  // codes 4kk, 4kk+1 of the run share a byte, and so do 4kk+2, 4kk+3
                                    const int wa = code_word_of<BITS>(ca), ba = code_byte_of<BITS>(ca), fa = code_field_of<BITS>(ca);
                                    const int wb = code_word_of<BITS>(cb), bb = code_byte_of<BITS>(cb), fb = code_field_of<BITS>(cb);
#pragma unroll
                                    for (int u = 0; u < MP; ++u) {
                                        uint32_t a0, a1, a2, a3;
                                        if constexpr (kSameView) {
                                            // slots (2t, 2t+1): channels 4kk, 4kk+2 (even nibbles of two bytes); (2t+8, 2t+9): 4kk+1, 4kk+3
                                            a0 = code_pair_same<BITS>(code_view<BITS, true>(w[u][0][wa], 0), ba, bb);
                                            a1 = code_pair_same<BITS>(code_view<BITS, true>(w[u][1][wa], 0), ba, bb);
                                            a2 = code_pair_same<BITS>(code_view<BITS, true>(w[u][0][wa], 1), ba, bb);
                                            a3 = code_pair_same<BITS>(code_view<BITS, true>(w[u][1][wa], 1), ba, bb);
                                        } else {
                                            a0 = code_pair<BITS>(code_view<BITS, false>(w[u][0][wa], fa), code_view<BITS, false>(w[u][0][wa], fa + 1), ba);
                                            a1 = code_pair<BITS>(code_view<BITS, false>(w[u][1][wa], fa), code_view<BITS, false>(w[u][1][wa], fa + 1), ba);
                                            a2 = code_pair<BITS>(code_view<BITS, false>(w[u][0][wb], fb), code_view<BITS, false>(w[u][0][wb], fb + 1), bb);
                                            a3 = code_pair<BITS>(code_view<BITS, false>(w[u][1][wb], fb), code_view<BITS, false>(w[u][1][wb], fb + 1), bb);
                                        }
                                        mma_16816<BF>(ch[u], a0, a1, a2, a3, b.x, b.y);
                                        mma_16816<BF>(cl[u], a0, a1, a2, a3, b.z, b.w);
                                    }
                                }
                            } else if (ip == 0) {  // a system-token unit is one tile
                                uint32_t w0[KC / 2], w1[KC / 2];  // the thread's KC channels of the two token rows, 16-bit pairs
                                lds_words_or_zero<KC / 2>(st + (g * D + KC * t) * (int)sizeof(CT), g < n_tok, w0);
                                lds_words_or_zero<KC / 2>(st + ((g + 8) * D + KC * t) * (int)sizeof(CT), g + 8 < n_tok, w1);
#pragma unroll
                                for (int kk = 0; kk < KS; ++kk) {
                                    const uint4 b = reinterpret_cast<const uint4 *>(xb)[kk * 32 + lane];
                                    mma_16816<CT>(ch[0], w0[2 * kk], w1[2 * kk], w0[2 * kk + 1], w1[2 * kk + 1], b.x, b.y);
                                    mma_16816<CT>(cl[0], w0[2 * kk], w1[2 * kk], w0[2 * kk + 1], w1[2 * kk + 1], b.z, b.w);
                                }
                            }
                        }
                        // base-2 scores; token slots without a token never win the maximum and weigh nothing
#pragma unroll
                        for (int u = 0; u < MP; ++u) {
                            const int r0 = (tile0 + ip + u) * 16 + g, r1 = r0 + 8;
                            sc[ip + u][0] = r0 < n_tok ? (ch[u][0] + cl[u][0] + bias_a) * p.scale_log2e : -INFINITY;
                            sc[ip + u][1] = r0 < n_tok ? (ch[u][1] + cl[u][1] + bias_b) * p.scale_log2e : -INFINITY;
                            sc[ip + u][2] = r1 < n_tok ? (ch[u][2] + cl[u][2] + bias_a) * p.scale_log2e : -INFINITY;
                            sc[ip + u][3] = r1 < n_tok ? (ch[u][3] + cl[u][3] + bias_b) * p.scale_log2e : -INFINITY;
                        }
                    }
                }

                // ---- phase 2: the warp's own online softmax.  New running maxima of query heads 2t, 2t + 1; the
                //      scores become weights in the warp's tile [head][token slot]; the running sums and outputs
                //      are rescaled when a maximum moved.
                float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
                for (int u = 0; u < MPW; ++u) {
                    mx_a = fmaxf(mx_a, fmaxf(sc[u][0], sc[u][2]));
                    mx_b = fmaxf(mx_b, fmaxf(sc[u][1], sc[u][3]));
                }
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, o));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, o));
                }
                const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);  // finite: the warp has a token
                if (__any_sync(0xffffffffu, mn_a > m_a || mn_b > m_b)) {
                    const float al_a = ex2(m_a - mn_a), al_b = ex2(m_b - mn_b);  // 0 on the warp's first unit
                    l_a *= al_a;
                    l_b *= al_b;
#pragma unroll
                    for (int mm = 0; mm < MT; ++mm) {
                        O[mm][0] *= al_a; O[mm][1] *= al_b; O[mm][2] *= al_a; O[mm][3] *= al_b;
                    }
                    m_a = mn_a;
                    m_b = mn_b;
                }
                float ws_a = 0.0f, ws_b = 0.0f;  // sums of this unit's weights of query heads 2t, 2t + 1
#pragma unroll
                for (int u = 0; u < MPW; ++u) {
                    const float w0 = ex2(sc[u][0] - mn_a), w1 = ex2(sc[u][1] - mn_b), w2 = ex2(sc[u][2] - mn_a), w3 = ex2(sc[u][3] - mn_b);
                    wt[(2 * t) * WP + 16 * u + g] = w0;
                    wt[(2 * t + 1) * WP + 16 * u + g] = w1;
                    wt[(2 * t) * WP + 16 * u + g + 8] = w2;
                    wt[(2 * t + 1) * WP + 16 * u + g + 8] = w3;
                    ws_a += w0 + w2;
                    ws_b += w1 + w3;
                }
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    ws_a += __shfl_xor_sync(0xffffffffu, ws_a, o);
                    ws_b += __shfl_xor_sync(0xffffffffu, ws_b, o);
                }
                l_a += ws_a;
                l_b += ws_b;
                __syncwarp();

                // ---- phase 3: this warp's share of the weighted sum of the values.  Rows of the product are
                //      channels: rows g and g + 8 of m-tile mm stand for channels VC*g + 2*mm and VC*g + 2*mm + 1; the
                //      contraction runs over the warp's tokens (slot 2t, 2t+1, 2t+8, 2t+9 of k-step ks is token 16 *
                //      (tile0 + ks) + the same); columns are query heads.  The accumulators start at minus the code
                //      offset times the sum of the weights, which takes the offset of the raw codes out again.
                //      d = 256 takes two passes of 8 m-tiles over the same weights.
                const unsigned char *vst = st + (is_sys ? kAtSysTokens * D * (int)sizeof(CT) : code_block);
#pragma unroll
                for (int m0 = 0; m0 < MT; m0 += MH) {
                    float acc[MH][4];
                    {
                        const float i_a = is_sys ? 0.0f : -kOff * ws_a, i_b = is_sys ? 0.0f : -kOff * ws_b;
#pragma unroll
                        for (int mm = 0; mm < MH; ++mm) {
                            acc[mm][0] = acc[mm][2] = i_a;
                            acc[mm][1] = acc[mm][3] = i_b;
                        }
                    }
#pragma unroll
                    for (int ks = 0; ks < MPW; ++ks) {
                        if (ks < n_tiles) {  // warp-uniform
                            const float2 wlo = *reinterpret_cast<const float2 *>(&wt[g * WP + 16 * ks + 2 * t]);
                            const float2 whi = *reinterpret_cast<const float2 *>(&wt[g * WP + 16 * ks + 2 * t + 8]);
                            uint32_t b0, b1, l0, l1;  // the weights, high and low parts
                            if (!is_sys) {
                                split2<BF>(wlo.x, wlo.y, b0, l0);
                                split2<BF>(whi.x, whi.y, b1, l1);
                                uint32_t w[4][(VB + 3) / 4];  // the thread's VC codes of its 4 tokens
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int tok = (tile0 + ks) * 16 + 2 * t + (e & 1) + 8 * (e >> 1);
                                    lds_code_bytes<VB>(vst + tok * p.g.row_bytes + g * VB, w[e]);
                                }
#pragma unroll
                                for (int mm = 0; mm < MH; ++mm) {
                                    // channels VC*g + 2*mm and the next one share a byte; rows g and g + 8 of the m-tile
                                    const int c = 2 * (m0 + mm);
                                    const int j = code_word_of<BITS>(c), b = code_byte_of<BITS>(c), f = code_field_of<BITS>(c);
                                    const uint32_t a0 = code_pair<BITS>(code_view<BITS, false>(w[0][j], f), code_view<BITS, false>(w[1][j], f), b);
                                    const uint32_t a1 = code_pair<BITS>(code_view<BITS, false>(w[0][j], f + 1), code_view<BITS, false>(w[1][j], f + 1), b);
                                    const uint32_t a2 = code_pair<BITS>(code_view<BITS, false>(w[2][j], f), code_view<BITS, false>(w[3][j], f), b);
                                    const uint32_t a3 = code_pair<BITS>(code_view<BITS, false>(w[2][j], f + 1), code_view<BITS, false>(w[3][j], f + 1), b);
                                    mma_16816<BF>(acc[mm], a0, a1, a2, a3, b0, b1);
                                    mma_16816<BF>(acc[mm], a0, a1, a2, a3, l0, l1);
                                }
                            } else if (ks == 0) {
                                split2<CT>(wlo.x, wlo.y, b0, l0);
                                split2<CT>(whi.x, whi.y, b1, l1);
                                uint32_t w[4][MH];  // the thread's channels VC*g + 2*(m0 + mm) (+1) of its 4 tokens, as 16-bit pairs
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int tok = 2 * t + (e & 1) + 8 * (e >> 1);
                                    lds_words_or_zero<MH>(vst + (tok * D + VC * g + 2 * m0) * (int)sizeof(CT), tok < n_tok, w[e]);
                                }
#pragma unroll
                                for (int mm = 0; mm < MH; ++mm) {
                                    const uint32_t a0 = __byte_perm(w[0][mm], w[1][mm], 0x5410), a1 = __byte_perm(w[0][mm], w[1][mm], 0x7632);
                                    const uint32_t a2 = __byte_perm(w[2][mm], w[3][mm], 0x5410), a3 = __byte_perm(w[2][mm], w[3][mm], 0x7632);
                                    mma_16816<CT>(acc[mm], a0, a1, a2, a3, b0, b1);
                                    mma_16816<CT>(acc[mm], a0, a1, a2, a3, l0, l1);
                                }
                            }
                        }
                    }
                    if (!is_sys) {
                        // acc holds sum_t w_t code_t: apply the group's scale and offset, channel by channel
                        const unsigned char *sv = st + 2 * code_block + 2 * meta_row, *mv = sv + meta_row;
#pragma unroll
                        for (int c8 = 0; c8 < 2 * MH / 8; ++c8) {
                            float s8[8], m8[8];
                            lds_meta8(sv, VC * g + 2 * m0 + c8 * 8, md, s8);
                            lds_meta8(mv, VC * g + 2 * m0 + c8 * 8, md, m8);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int mm = c8 * 4 + j;
                                O[m0 + mm][0] = fmaf(s8[2 * j], acc[mm][0], fmaf(m8[2 * j], ws_a, O[m0 + mm][0]));
                                O[m0 + mm][1] = fmaf(s8[2 * j], acc[mm][1], fmaf(m8[2 * j], ws_b, O[m0 + mm][1]));
                                O[m0 + mm][2] = fmaf(s8[2 * j + 1], acc[mm][2], fmaf(m8[2 * j + 1], ws_a, O[m0 + mm][2]));
                                O[m0 + mm][3] = fmaf(s8[2 * j + 1], acc[mm][3], fmaf(m8[2 * j + 1], ws_b, O[m0 + mm][3]));
                            }
                        }
                    } else {
#pragma unroll
                        for (int mm = 0; mm < MH; ++mm)
#pragma unroll
                            for (int e = 0; e < 4; ++e) O[m0 + mm][e] += acc[mm][e];
                    }
                }
                __syncwarp();  // every lane is done with the weight tile (and, a team of one warp, with the stage)
            }
            if (TW == 1 && i + S < n_mine && !dead) {  // a team of one: its stage is free the moment the unit is done
                const int in = i + S;
                const int32_t tb = (in >> 5) == (i >> 5) ? tg_batch : load_tg_batch(in & ~31);
                post_unit(in, s, __shfl_sync(0xffffffffu, tb, in & 31));
            }
            if (((i + 1) & 31) == 0 && i + 1 < n_mine) tg_batch = load_tg_batch(i + 1);
            s_prev = s;
            s = s + 1 == S ? 0 : s + 1;
        }

        // ---- merge the warps of the block.  Each warp rescales its output to the block's maximum and parks it in the
        //      ring (free by now), laid out so that neither these stores nor the sums below collide on banks.
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
        // nothing may still be landing in the ring when it takes the results (only after a wait ran out)
        for (int z = 0; z < S; ++z) {
            if ((stage_info >> (8 * z)) & 0x7Fu) {
                mbar_wait_bounded(bar0 + 8 * z, (phase_bits >> z) & 1u, abort_flag + 1, kAtWaitLimitNs);
                phase_bits ^= 1u << z;
                stage_info &= ~(0xFFu << (8 * z));
            }
        }
        __syncthreads();
        {
            float M_a = -INFINITY, M_b = -INFINITY;
            for (int w = 0; w < n_warps; ++w) {
                M_a = fmaxf(M_a, stat[w * 16 + 2 * t]);
                M_b = fmaxf(M_b, stat[w * 16 + 2 * t + 1]);
            }
            const float f_a = m_a == -INFINITY ? 0.0f : ex2(m_a - M_a), f_b = m_b == -INFINITY ? 0.0f : ex2(m_b - M_b);
            float *mine = reinterpret_cast<float *>(ring) + warp * (8 * D);
#pragma unroll
            for (int mm = 0; mm < MT; ++mm) {
                *reinterpret_cast<float2 *>(mine + at_oidx<VC>(g, 2 * mm, 2 * t)) = make_float2(O[mm][0] * f_a, O[mm][1] * f_b);
                *reinterpret_cast<float2 *>(mine + at_oidx<VC>(g, 2 * mm + 1, 2 * t)) = make_float2(O[mm][2] * f_a, O[mm][3] * f_b);
            }
        }
        __syncthreads();
        for (int e = tid; e < 8 * D; e += n_threads) {
            float a = 0.0f;
            for (int w = 0; w < n_warps; ++w) a += reinterpret_cast<const float *>(ring)[w * (8 * D) + e];
            ob[e] = a;
        }
        if (tid < kAtHeads) {
            float M = -INFINITY, L = 0.0f;
            for (int w = 0; w < n_warps; ++w) M = fmaxf(M, stat[w * 16 + tid]);
            for (int w = 0; w < n_warps; ++w) {
                const float mw = stat[w * 16 + tid];
                if (mw != -INFINITY) L = fmaf(stat[w * 16 + 8 + tid], ex2(mw - M), L);
            }
            blk[tid] = M;
            blk[8 + tid] = L;
        }

        // ---- merge the blocks of the cluster: rank r finishes its share of the (channel, head) pairs
        if (C > 1) cluster_sync(); else __syncthreads();
        {
            const int per = (8 * D + (int)C - 1) / (int)C;
            const int e_end = min(per * ((int)r + 1), 8 * D);
            for (int e = per * (int)r + tid; e < e_end; e += n_threads) {
                const int slab = e / (VC * 8), rem = e - slab * (VC * 8);
                const int hh = rem & 7, cl = ((rem >> 3) - slab + VC) % VC;
                if (hh >= nh) continue;  // a head beyond the GQA block
                float num = 0.0f, den = 0.0f;
                if (C > 1) {
                    // every block's (max, sum, partial) of this pair is asked for before any of them is used
                    float Mb[kAtMaxCluster], Lb[kAtMaxCluster], Ov[kAtMaxCluster];
#pragma unroll
                    for (uint32_t b = 0; b < kAtMaxCluster; ++b) {
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
                    for (int b = 0; b < kAtMaxCluster; ++b) M = fmaxf(M, Mb[b]);
#pragma unroll
                    for (int b = 0; b < kAtMaxCluster; ++b) {
                        const float f = Mb[b] == -INFINITY ? 0.0f : ex2(Mb[b] - M);
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

static int attend_units(int32_t k, int32_t sys_len, int *n_sys_units) {
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

// One way to run the kernel: warps per team, teams per block, ring depth, and what the device holds of it
struct AttendShape {
    int teams = 0, stages = 0;
    size_t smem = 0;
    int clusters[kAtMaxCluster + 1] = {};  // clusters of c blocks resident at once (0: cannot be launched)
};
// What the driver said about the shapes of one kernel instantiation; asked once per process and device.
struct AttendResidency {
    std::mutex mu;
    int dev = -1, stage_bytes = 0, sms = 0, n_shapes = 0;
    AttendShape shapes[3];
};

// Fills `res` for the instantiation `kernel` (MPW fixed): the candidate block shapes and their residency.
template <typename KernelT>
static cudaError_t attend_probe(KernelT kernel, AttendResidency &res, int dev, int D, int MPW, int stage_bytes) {
    int smem_max = 0;
    cudaError_t e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&res.sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    const int TW = 4 / MPW;
    res.n_shapes = 0;
    // as many teams as a block of 16 warps has, fewer if their rings (two stages at least where a team has several
    // warps) do not fit beside each other; then as deep a ring as fits
    int cand[1], n_cand = 0;
    {
        int most = kAtMaxWarps / TW;
        while (most > 1 && at_layout(D, MPW, most, TW > 1 ? 2 : 1, stage_bytes).total > smem_max) --most;
        cand[n_cand++] = most;
    }
    for (int ci = 0; ci < n_cand; ++ci) {
        AttendShape &sh = res.shapes[res.n_shapes];
        sh.teams = cand[ci];
        sh.stages = TW > 1 ? kAtMaxStages : 1;
        while (sh.stages > (TW > 1 ? 2 : 1) && at_layout(D, MPW, sh.teams, sh.stages, stage_bytes).total > smem_max) --sh.stages;
        sh.smem = (size_t)at_layout(D, MPW, sh.teams, sh.stages, stage_bytes).total;
        if ((int)sh.smem > smem_max) continue;
        cudaLaunchConfig_t lc = {};
        lc.blockDim = dim3(sh.teams * TW * 32);
        lc.dynamicSmemBytes = sh.smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        lc.attrs = at;
        lc.numAttrs = 1;
        for (int c = 1; c <= kAtMaxCluster; ++c) {
            lc.gridDim = dim3((unsigned)c, 1, 1);
            at[0].val.clusterDim.x = (unsigned)c;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kernel, &lc) != cudaSuccess) {
                (void)cudaGetLastError();
                n = 0;
            }
            sh.clusters[c] = n;
        }
        ++res.n_shapes;
    }
    res.dev = dev;
    res.stage_bytes = stage_bytes;
    return cudaSuccess;
}

// Estimated run time (microseconds, roughly) of `pairs` (layer, kv head) pairs of `units` units each (n_sys of them
// short ones) on clusters of c blocks of `teams` teams: waves of resident clusters x (fixed cost of a block + the
// longest walk of a team x the time a team takes over a unit).
static double attend_cost(const AttendShape &sh, int c, int64_t pairs, int units, int n_sys, double fixed, double unit_time) {
    if (sh.clusters[c] < 1) return 1e30;
    const int teams = c * sh.teams;
    if (c > 1 && (c - 1) * sh.teams >= units) return 1e30;  // the last block would have nothing to do
    // team tm walks units tm, tm + teams, ...; the first n_sys units are system-token units (about a third of a group)
    double worst = 0.0;
    for (int tm = 0; tm < teams && tm < units; ++tm) {
        const int n = (units - tm + teams - 1) / teams;
        const int sys = tm < n_sys ? (n_sys - tm + teams - 1) / teams : 0;
        const double load = (n - sys) + 0.3 * sys;
        if (load > worst) worst = load;
    }
    const double waves = (double)((pairs + sh.clusters[c] - 1) / sh.clusters[c]);
    return waves * (fixed + worst * unit_time) + 0.02 * c;
}

struct AttendPlan {
    double cost = 1e30;
    int shape = -1, c = 0;
};
static AttendPlan attend_plan(const AttendResidency &res, int64_t pairs, int units, int n_sys, double fixed, double unit_time) {
    AttendPlan best;
    for (int si = 0; si < res.n_shapes; ++si)
        for (int c = 1; c <= kAtMaxCluster; ++c) {
            const double cost = attend_cost(res.shapes[si], c, pairs, units, n_sys, fixed, unit_time);
            if (cost < best.cost) {
                best.cost = cost;
                best.shape = si;
                best.c = c;
            }
        }
    return best;
}

template <typename KernelT>
static int32_t attend_launch(KernelT kernel, const AttendResidency &res, const AttendPlan &plan, const AttendParams &p,
                             int MPW, int layers, cudaStream_t s) {
    const AttendShape &sh = res.shapes[plan.shape];
    AttendParams q = p;
    q.teams = sh.teams;
    q.n_stages = sh.stages;
    cudaLaunchConfig_t lc = {};
    lc.blockDim = dim3(sh.teams * (4 / MPW) * 32);
    lc.dynamicSmemBytes = sh.smem;
    lc.stream = s;
    lc.gridDim = dim3((unsigned)plan.c, (unsigned)p.g.H, (unsigned)layers);
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)plan.c;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see the kernel's prologue
    at[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&lc, kernel, q);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    return finish_launch();
}

// Both shapes of the kernel for one combination of types: the plan with the shorter estimate runs.  Measured on
// B200: a block of four-warp teams costs about 6 us before and after its units and a team takes about 3.2 us over a
// group; a block of two-warp teams costs about 7 us and a team takes about 4.3 us over a group with the multiprocessor
// full of them (8 teams against 4).
template <typename QT, typename CT, int D, int BITS>
static int32_t launch_attend_inst(const AttendParams &p, int layers, cudaStream_t s) {
    static AttendResidency res1, res2;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) {
        std::lock_guard<std::mutex> lock(res1.mu);
        if (res1.dev != dev || res1.stage_bytes != p.stage_bytes) {
            e = attend_probe(attend_kernel<QT, CT, D, BITS, 1>, res1, dev, D, 1, p.stage_bytes);
            if (e == cudaSuccess) e = attend_probe(attend_kernel<QT, CT, D, BITS, 2>, res2, dev, D, 2, p.stage_bytes);
        }
    }
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    const int64_t pairs = (int64_t)p.g.H * layers;
    const AttendPlan p1 = attend_plan(res1, pairs, p.n_units, p.n_sys_units, 6.0, 3.2);
    const AttendPlan p2 = attend_plan(res2, pairs, p.n_units, p.n_sys_units, 7.2, 4.3);
    if (p1.shape < 0 && p2.shape < 0) return STOM_ERR_SHAPE;
    if (p1.cost <= p2.cost) return attend_launch(attend_kernel<QT, CT, D, BITS, 1>, res1, p1, p, 1, layers, s);
    return attend_launch(attend_kernel<QT, CT, D, BITS, 2>, res2, p2, p, 2, layers, s);
}

template <typename QT, typename CT>
static int32_t launch_attend(const AttendParams &p, int layers, cudaStream_t s) {
    const bool b4 = p.g.row_bytes * 2 == p.g.d;  // 4-bit codes: d/2 bytes per row
    switch (p.g.d) {
    case 64: return b4 ? launch_attend_inst<QT, CT, 64, 4>(p, layers, s) : launch_attend_inst<QT, CT, 64, 2>(p, layers, s);
    case 128: return b4 ? launch_attend_inst<QT, CT, 128, 4>(p, layers, s) : launch_attend_inst<QT, CT, 128, 2>(p, layers, s);
    case 256: return b4 ? launch_attend_inst<QT, CT, 256, 4>(p, layers, s) : launch_attend_inst<QT, CT, 256, 2>(p, layers, s);
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
    p.n_units = attend_units(k, sys_len, &p.n_sys_units);
    p.stage_bytes = attend_stage_bytes(cfg);
    p.n_stages = 1;
    p.teams = 1;
    p.scale_log2e = softmax_scale * 1.4426950408889634f;
    p.flags = dev_flags;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (layer_count > 65535 || cfg->n_kv_heads > 65535) return STOM_ERR_SHAPE;
    const bool bf = cache_dtype == STOM_BF16;
    switch (cfg->kv_dtype) {
    case STOM_BF16:
        return bf ? launch_attend<__nv_bfloat16, __nv_bfloat16>(p, layer_count, s)
                  : launch_attend<__nv_bfloat16, __half>(p, layer_count, s);
    case STOM_FP16:
        return bf ? launch_attend<__half, __nv_bfloat16>(p, layer_count, s)
                  : launch_attend<__half, __half>(p, layer_count, s);
    default:
        return bf ? launch_attend<float, __nv_bfloat16>(p, layer_count, s)
                  : launch_attend<float, __half>(p, layer_count, s);
    }
}
