// A1: group quantizer + representative key (paper Sec. 3.4: Q_4, (s_t, m_t),
// k-bar; appendix "Layer-wise vision memory").
//
// A tile is the G tokens x d channels of one (layer, frame, kv head) of K or
// of V (12.8 KB at G = 50, d = 128, bf16).  The kernel is persistent: one
// block per SM, up to kConsumerWarps consumer warps and one producer warp.
//
//   producer  walks the block's tiles and, for each, issues bulk asynchronous
//             copies (cp.async.bulk, completion counted on an mbarrier) from
//             global memory into a ring of shared-memory slots that fills
//             the SM's shared memory (18 slots at 12.8 KB): tile n goes to
//             slot n % N.  A tile whose rows are contiguous is one copy, and
//             the lanes of the warp each look after one slot of a group of N
//             consecutive tiles, filling it the moment its consumer lets go;
//             a strided or index-gathered tile is one copy per row, issued
//             by the whole warp tile after tile.  Whatever is not being read
//             by a consumer is in flight, which is what hides HBM latency;
//             no register is tied up by a load.
//   consumer  warp w takes every n_warps-th tile of the block outright.
//             A lane owns d/32 adjacent channels of ALL G rows, so the
//             per-channel statistics need no cross-lane traffic at all:
//               pass 1  packed min / max down the rows (shared memory reads)
//               stats   s = (max - min)/15, m = min, y = rn(1/s)   -> global
//               pass 2  codes, two channels per instruction (f32x2), stored
//                       straight to the bank (a warp's store covers one
//                       packed row); key tiles add up the rows for the
//                       representative key on the way
//             Sixteen such warps keep the issue slots busy while each one
//             sits out the fixed latencies of its own division chains.
//
// Every wait on an mbarrier is bounded (wall-clock limit); a wait that runs
// out sets STOM_FLAG_TIMEOUT, tells the rest of the block to stop, and the
// block drains its copies in flight before it returns.
//
// Bit-exactness of the codes: the contract is code = rne(fl((x - m) / s)) in
// binary32 with a true division.  A hardware-exact division per element would
// make the kernel instruction-bound, so the quotient is formed with the
// correctly rounded reciprocal y = rn(1/s), its remainder y_lo = rn(1/s - y)
// (both per channel, once per tile) and one residual correction
//     q0 = rn(diff*y + rn(diff*y_lo)); e = rn(diff - q0*s); q1 = rn(q0 + e*y)
// (y + y_lo carries 1/s to about 47 bits, so q0 is within half an ulp of the
// quotient up to 2^-22 ulp: a faithful quotient; and a faithful quotient
// corrected once with an exact FMA residual and a correctly rounded reciprocal
// is the correctly rounded quotient -- Markstein's division theorem), followed
// by the add-magic-constant trick for round-half-even.  That is six packed
// operations per pair of channels; starting from rn(diff*y) alone, which is
// not always faithful, took two corrections and seven.  Tiles with a channel whose
// scale is zero or outside (2^-60, 2^60) take a slow path with the IEEE division.
#include "stom_async.cuh"
#include "stom_internal.cuh"

namespace stom {

constexpr int kConsumerWarps = 16;
constexpr int kQuantThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxSlots = 32;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s: far beyond any legitimate wait

struct QuantParams {
    const void *K, *V, *Ksum;
    const int32_t *token_idx;
    int64_t sl, sg, sh, st;  // element strides: layer, group(frame), head, token
    uint8_t *codes_k, *codes_v;
    void *scale_k, *zero_k, *scale_v, *zero_v, *rep_key;  // elements of g.meta_dtype
    float *rep_norm2;
    BankGeom g;
    int32_t layer_begin, group_begin, F, n_in;
    uint32_t *flags;
    uint32_t n_tiles;     // layer_count * F * H * n_kinds, below 2^31
    int32_t n_kinds;      // 2: keys, values;  3: keys, values, pre-rotary keys (mean only)
    int32_t n_slots;      // ring depth
    int32_t n_warps;      // consumer warps that take tiles, at most n_slots (the others leave at once)
    int32_t slot_bytes;   // bytes of one input tile, rounded up to 128
    int32_t contiguous;   // rows of a tile are adjacent in global memory
};

// Bounded wait on an mbarrier (stom_async.cuh has the wrappers).  Returns false when the limit ran out or another
// thread of the block gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag) {
    return mbar_wait_bounded(bar, parity, abort_flag, kWaitLimitNs);
}

// ------------------------------------------------------------------ arithmetic

// IEEE division; s == 0 marks a constant (or underflowing) channel whose codes are all 0
__device__ __forceinline__ uint32_t code_slow(float x, float m, float s, float levels) {
    if (s == 0.0f) return 0u;
    const float t = __fdiv_rn(__fsub_rn(x, m), s);
    float r = rintf(t);
    r = fminf(fmaxf(r, 0.0f), levels);
    return (uint32_t)r;
}

// element-wise min / max on one 32-bit word of a row (two 16-bit values or one float)
template <typename T> struct WordOps;
template <> struct WordOps<__nv_bfloat16> {
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

// Two adjacent channels at once: x - m, the correctly rounded quotient, the rounding add.  Returns the two floats
// 1.5*2^23 + code as a pair.  y = rn(1/s) and y_lo = rn(1/s - y) together carry 1/s to about 47 bits, so
// q0 = rn(diff*y + rn(diff*y_lo)) is within 0.5 ulp (plus 2^-22 ulp) of diff/s: a faithful quotient, which one
// correction with the exact FMA residual turns into the correctly rounded one.
__device__ __forceinline__ uint64_t code_pair(uint64_t x, uint64_t m, uint64_t neg_s, uint64_t y, uint64_t y_lo,
                                              uint64_t magic) {
    const uint64_t diff = sub2(x, m);
    uint64_t q = fma2(diff, y, mul2(diff, y_lo));
    const uint64_t e = fma2(q, neg_s, diff);
    q = fma2(e, y, q);
    return add2(q, magic);
}

// The C channels of one token row that a lane owns, as 32-bit words read from shared memory.
template <typename T, int C>
struct LaneRow {
    static constexpr int W = C * (int)sizeof(T) / 4;
    uint32_t w[W];
    __device__ __forceinline__ void load(const unsigned char *p) {
        if constexpr (W == 1) {
            w[0] = *reinterpret_cast<const uint32_t *>(p);
        } else if constexpr (W == 2) {
            const uint2 v = *reinterpret_cast<const uint2 *>(p);
            w[0] = v.x; w[1] = v.y;
        } else {
#pragma unroll
            for (int i = 0; i < W / 4; ++i) {
                const uint4 v = *reinterpret_cast<const uint4 *>(p + 16 * i);
                w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
            }
        }
    }
    // channels 2j and 2j+1 as floats (exact)
    __device__ __forceinline__ void pair(int j, float &a, float &b) const {
        if constexpr (sizeof(T) == 4) {
            a = __uint_as_float(w[2 * j]);
            b = __uint_as_float(w[2 * j + 1]);
        } else {
            unpack2<T>(w[j], a, b);
        }
    }
};

template <int C>
__device__ __forceinline__ void store_floats(float *dst, const float (&v)[C]) {
    if constexpr (C == 2) {
        *reinterpret_cast<float2 *>(dst) = make_float2(v[0], v[1]);
    } else {
#pragma unroll
        for (int i = 0; i < C; i += 4) *reinterpret_cast<float4 *>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
    }
}

// ---- 16-bit metadata.  The stored offset must not exceed the channel minimum and the stored scale must reach the
// channel maximum from it, so the offset rounds towards -inf and the scale towards +inf; the codes are then taken
// against the stored pair.  bfloat16 is the upper half of a binary32: truncation rounds towards zero, one step more
// on the side that needs it.  binary16 has conversion instructions with both directed modes.
__device__ __forceinline__ float meta_round_down(float x, int meta_dtype) {
    if (meta_dtype == STOM_BF16) {
        const uint32_t u = __float_as_uint(x);
        return __uint_as_float((u & 0xffff0000u) + (((u & 0xffffu) != 0u && (u >> 31)) ? 0x10000u : 0u));
    }
    return __half2float(__float2half_rd(x));
}
__device__ __forceinline__ float meta_round_up(float x, int meta_dtype) {
    if (meta_dtype == STOM_BF16) {
        const uint32_t u = __float_as_uint(x);
        return __uint_as_float((u & 0xffff0000u) + (((u & 0xffffu) != 0u && !(u >> 31)) ? 0x10000u : 0u));
    }
    return __half2float(__float2half_ru(x));
}
__device__ __forceinline__ float meta_round_nearest(float x, int meta_dtype) {
    return meta_dtype == STOM_BF16 ? __bfloat162float(__float2bfloat16_rn(x)) : __half2float(__float2half_rn(x));
}

// C adjacent metadata values to element `at` of a bank array of type meta_dtype; for the 16-bit types the values are
// already representable, so the conversion is exact.
template <int C>
__device__ __forceinline__ void store_meta(void *base, int64_t at, int meta_dtype, const float (&v)[C]) {
    if (meta_dtype == STOM_FP32) {
        store_floats<C>(static_cast<float *>(base) + at, v);
        return;
    }
    uint32_t w[C / 2];
#pragma unroll
    for (int i = 0; i < C / 2; ++i)
        w[i] = meta_dtype == STOM_BF16 ? pack2<__nv_bfloat16>(v[2 * i], v[2 * i + 1]) : pack2<__half>(v[2 * i], v[2 * i + 1]);
    uint16_t *dst = static_cast<uint16_t *>(base) + at;
    if constexpr (C == 2) *reinterpret_cast<uint32_t *>(dst) = w[0];
    else if constexpr (C == 4) *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1]);
    else *reinterpret_cast<uint4 *>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
}

// The C * BITS code bits of one row that a lane produced go to dst = row start + byte offset of the lane.  With
// 2 channels of 2 bits a lane has only half a byte: the even lane takes its neighbour's half and stores for both.
template <int C, int BITS>
__device__ __forceinline__ void store_codes(unsigned char *dst, uint32_t cw, int lane) {
    constexpr int NB = C * BITS;
    if constexpr (NB == 4) {
        const uint32_t hi = __shfl_down_sync(0xffffffffu, cw, 1);
        if (!(lane & 1)) *dst = (unsigned char)((cw & 15u) | (hi << 4));
    } else if constexpr (NB == 8) {
        *dst = (unsigned char)cw;
    } else if constexpr (NB == 16) {
        *reinterpret_cast<uint16_t *>(dst) = (uint16_t)cw;
    } else {
        *reinterpret_cast<uint32_t *>(dst) = cw;
    }
}

// Pass 2 on the fast path: the codes of this lane's C channels for all G rows of a tile, written to the staging
// tile; SUM also adds the rows up (keys: the representative key is their mean).
template <typename T, int C, int BITS, bool SUM>
__device__ __forceinline__ void code_rows(const unsigned char *tile, unsigned char *out_lane, int G, int lane,
                                          const uint64_t (&m2)[C / 2], const uint64_t (&ns2)[C / 2],
                                          const uint64_t (&y2)[C / 2], const uint64_t (&yl2)[C / 2],
                                          uint64_t (&sum2)[C / 2]) {
    constexpr int ROW_BYTES = 32 * C * (int)sizeof(T), CODE_ROW = 4 * C * BITS;
    const uint64_t magic = pack_f2(12582912.0f, 12582912.0f);  // 1.5 * 2^23: rounds to integer, ties to even
    // every float 1.5*2^23 + code has the bit pattern 0x4B400000 + code; summing pattern << (BITS * channel) over
    // the lane's channels leaves the codes in place in the low BITS*C bits (they cannot carry into each other);
    // only with 8 channels of 4 bits does the constant part wrap into the word, and it is removed up front
    constexpr uint32_t kBias = (C == 8 && BITS == 4) ? 0x4B400000u * 0x11111111u : 0u;
    auto code_word = [&](const LaneRow<T, C> &row) -> uint32_t {
        uint32_t cw = 0u - kBias;
#pragma unroll
        for (int j = 0; j < C / 2; ++j) {
            float x0, x1;
            row.pair(j, x0, x1);
            const uint64_t x = pack_f2(x0, x1);
            if constexpr (SUM) sum2[j] = add2(sum2[j], x);
            const uint64_t u = code_pair(x, m2[j], ns2[j], y2[j], yl2[j], magic);
            float u0, u1;
            unpack_f2(u, u0, u1);
            cw += __float_as_uint(u0) << (2 * BITS * j);
            cw += __float_as_uint(u1) << (2 * BITS * j + BITS);
        }
        return cw;
    };
    // Rows go through in batches: all loads of a batch, then its arithmetic, then its stores.  The compiler cannot
    // prove that the staging tile and the input tile do not overlap, so a load would never move above an earlier
    // store; batching by hand gives it kBatch * C/2 independent division chains to interleave.
    constexpr int kBatch = C == 8 ? 3 : 5;
    int r = 0;
    for (; r + kBatch <= G; r += kBatch) {
        LaneRow<T, C> rows[kBatch];
        uint32_t cw[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) rows[i].load(tile + (r + i) * ROW_BYTES);
#pragma unroll
        for (int i = 0; i < kBatch; ++i) cw[i] = code_word(rows[i]);
#pragma unroll
        for (int i = 0; i < kBatch; ++i) store_codes<C, BITS>(out_lane + (r + i) * CODE_ROW, cw[i], lane);
    }
    for (; r < G; ++r) {
        LaneRow<T, C> row;
        row.load(tile + r * ROW_BYTES);
        store_codes<C, BITS>(out_lane + r * CODE_ROW, code_word(row), lane);
    }
}

// ------------------------------------------------------------------ tile bookkeeping

struct TileCoord {
    int kind, h, f, li;
};
__device__ __forceinline__ TileCoord tile_coord(uint32_t tau, const QuantParams &p) {
    TileCoord t;
    t.kind = (int)(tau % (uint32_t)p.n_kinds);
    tau /= (uint32_t)p.n_kinds;
    t.h = (int)(tau % (uint32_t)p.g.H);
    tau /= (uint32_t)p.g.H;
    t.f = (int)(tau % (uint32_t)p.F);
    t.li = (int)(tau / (uint32_t)p.F);
    return t;
}

// What the producer tells the consumer about the tile it put into a ring slot.
struct SlotInfo {
    int64_t bslot;  // index of (layer, group, head) in the bank
    int32_t kind;   // 0 keys, 1 values, 2 pre-rotary keys
    int32_t round;  // fill number of the slot's latest fill, -1 before the first (read by the producer's final drain)
};

// shared memory: [full[2][kMaxSlots], empty[kMaxSlots]] [abort words] [SlotInfo[kMaxSlots]] [ring of input slots]
constexpr int kAbortOff = 3 * kMaxSlots * 8;
constexpr int kInfoOff = 1024;
constexpr int kBarBytes = 2048;
static_assert(kAbortOff + 8 <= kInfoOff && kInfoOff + kMaxSlots * (int)sizeof(SlotInfo) <= kBarBytes, "header layout");

// C: channels per lane (d / 32).  blockDim.x = kQuantThreads, one block per SM, grid-stride over tiles.
// MD: type the bank keeps s, m and k-bar in (STOM_FP32 | STOM_FP16 | STOM_BF16)
template <typename T, int C, int BITS, int MD>
__global__ void __launch_bounds__(kQuantThreads, 1) quantize_kernel(const QuantParams p) {
    constexpr float kLevels = (float)((1 << BITS) - 1);  // 15 levels above the offset at 4 bits, 3 at 2 bits
    constexpr int D = 32 * C;
    constexpr int LANE_BYTES = C * (int)sizeof(T);  // bytes of a row that one lane owns
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int CODE_ROW = D * BITS / 8;          // packed bytes per token row
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kAbortOff);
    SlotInfo *info = reinterpret_cast<SlotInfo *>(smem + kInfoOff);
    unsigned char *ring = smem + kBarBytes;
    const int G = p.g.G, N = p.n_slots;
    const uint32_t tile_bytes = (uint32_t)G * ROW_BYTES;
    const uint32_t code_bytes = (uint32_t)G * CODE_ROW;
    // Tile n of the block goes to ring slot n % N and to consumer warp n % n_warps.  A slot has TWO "full" barriers
    // used by alternate fills: a waiter only tells a barrier's phases apart by one parity bit, and with a single
    // barrier a warp that runs ahead could take fill k-1 of its slot, still on its way, for fill k.  With two, the
    // fill it could be confused with is k-2; the consumer rules that out by the fill number the producer publishes
    // in the slot's info record before it starts a copy (see the consumers' wait).  The fills of ONE slot are issued
    // in order and each waits for the release of the one before, so one "empty" barrier per slot is enough.
    const uint32_t WA = (uint32_t)p.n_warps;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 2 * kMaxSlots * 8;
    auto full_bar = [&](int slot, uint32_t round) -> uint32_t { return full0 + 8 * ((round & 1u) * kMaxSlots + slot); };

    // The launch may overlap the tail of the kernel ahead of it in the stream (programmatic dependent launch): the
    // barriers are set up meanwhile, and every thread waits for that kernel before it touches global memory.
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < N; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(full0 + 8 * (kMaxSlots + i), 1);
            mbar_init(empty0 + 8 * i, 1);
            info[i].round = -1;
        }
        abort_flag[0] = 0;  // set by the first thread whose wait ran out
        abort_flag[1] = 0;  // never set: lets the final drain wait regardless of an abort
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    grid_dependency_wait();  // the frames may come from, and the bank may still be read by, the kernel just ahead

    // tiles of this block: tau = blockIdx.x + n * gridDim.x, n = 0 .. my_count-1
    const uint32_t my_count = p.n_tiles > blockIdx.x ? (p.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;

    if (warp == kConsumerWarps) {
        // =============================================================== producer
        bool stop = false;
        if (p.contiguous) {
            // One bulk copy per tile.  Issued tile by tile by one thread, a tile cost the warp about 500 cycles of
            // dependent instructions (wait, publish, expect, copy) and the whole block no more than one tile per
            // 0.3 us, whatever the consumers did.  So a group of up to N consecutive tiles -- N ring slots, each
            // slot at most once -- is handled by N lanes at once: every lane polls (without blocking) whether its
            // own slot has been released and fills it the moment it has, in whatever order the slots come free.
            // Groups follow one another, so the fills of one slot are still issued in order; what is lost is the
            // order BETWEEN slots, which the consumers make up for (see their wait).
            int slot0 = 0;        // slot of the group's first tile
            uint32_t round0 = 0;  // and its fill number
            for (uint32_t n0 = 0; n0 < my_count && !stop; n0 += (uint32_t)N) {
                const int cnt = (int)(my_count - n0 < (uint32_t)N ? my_count - n0 : (uint32_t)N);
                bool pending = lane < cnt;
                int my_slot = slot0 + lane;
                uint32_t my_round = round0;
                if (my_slot >= N) {
                    my_slot -= N;
                    ++my_round;
                }
                TileCoord tl = {0, 0, 0, 0};
                const T *src = nullptr;
                int64_t bslot = 0;
                if (pending) {
                    tl = tile_coord(blockIdx.x + (n0 + lane) * gridDim.x, p);
                    src = reinterpret_cast<const T *>(tl.kind == 0 ? p.K : (tl.kind == 1 ? p.V : p.Ksum)) +
                          (int64_t)tl.li * p.sl + (int64_t)tl.f * p.sg + (int64_t)tl.h * p.sh;
                    bslot = bank_slot(p.g, p.layer_begin + tl.li, p.group_begin + tl.f, tl.h);
                }
                unsigned long long t0 = 0;
                for (uint32_t spin = 0;; ++spin) {
                    if (pending && (my_round == 0 || mbar_test(empty0 + 8 * my_slot, (my_round - 1) & 1u))) {
                        info[my_slot].bslot = bslot;  // published by the release of the arrive below
                        info[my_slot].kind = tl.kind;
                        info[my_slot].round = (int32_t)my_round;
                        const uint32_t bar = full_bar(my_slot, my_round);
                        mbar_expect_tx(bar, tile_bytes);
                        bulk_load(smem_u32(ring + (size_t)my_slot * p.slot_bytes), src, tile_bytes, bar);
                        pending = false;
                    }
                    if (!__any_sync(0xffffffffu, pending)) break;
                    if ((spin & 63u) == 63u) {  // bounded: a slot that never comes free ends the block
                        if (t0 == 0) t0 = global_ns();
                        if (__any_sync(0xffffffffu, *abort_flag || global_ns() - t0 > kWaitLimitNs)) {
                            if (lane == 0) {
                                if (!*abort_flag && p.flags) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
                                *abort_flag = 1;
                            }
                            stop = true;
                            break;
                        }
                    }
                }
                slot0 += cnt;
                if (slot0 >= N) {
                    slot0 -= N;
                    ++round0;
                }
            }
        } else {
            // Rows of a tile are strided or picked by token_idx: one bulk copy per row, the warp's lanes sharing out
            // the rows of one tile at a time.  Tile coordinates cost a few integer divisions, so the 32 lanes work
            // out 32 consecutive tiles at once and hand the results round by shuffle.
            int slot = 0;
            uint32_t round = 0;  // fill number of `slot`
            for (uint32_t n0 = 0; n0 < my_count && !stop; n0 += 32) {
                const uint32_t mine = n0 + lane < my_count ? n0 + lane : my_count - 1;
                const TileCoord tl = tile_coord(blockIdx.x + mine * gridDim.x, p);
                const unsigned long long src_l = reinterpret_cast<unsigned long long>(
                    reinterpret_cast<const T *>(tl.kind == 0 ? p.K : (tl.kind == 1 ? p.V : p.Ksum)) +
                    (int64_t)tl.li * p.sl + (int64_t)tl.f * p.sg + (int64_t)tl.h * p.sh);
                const long long bslot_l = bank_slot(p.g, p.layer_begin + tl.li, p.group_begin + tl.f, tl.h);
                const int cnt = (int)(my_count - n0 < 32u ? my_count - n0 : 32u);
                for (int i = 0; i < cnt; ++i) {
                    bool ok = true;
                    if (round > 0) ok = mbar_wait(empty0 + 8 * slot, (round - 1) & 1u, abort_flag);
                    ok = __all_sync(0xffffffffu, ok && !*abort_flag);  // the whole warp stops together
                    if (!ok) {
                        if (lane == 0) {
                            if (!*abort_flag && p.flags) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
                            *abort_flag = 1;
                        }
                        stop = true;
                        break;
                    }
                    const T *src = reinterpret_cast<const T *>(__shfl_sync(0xffffffffu, src_l, i));
                    const long long bslot = __shfl_sync(0xffffffffu, bslot_l, i);
                    const int kind = __shfl_sync(0xffffffffu, tl.kind, i);
                    const int f = __shfl_sync(0xffffffffu, tl.f, i);
                    const uint32_t bar = full_bar(slot, round);
                    const uint32_t dst = smem_u32(ring + (size_t)slot * p.slot_bytes);
                    if (lane == 0) {
                        info[slot].bslot = bslot;  // published by the release of the arrive below
                        info[slot].kind = kind;
                        info[slot].round = (int32_t)round;
                        mbar_expect_tx(bar, tile_bytes);
                    }
                    __syncwarp();
                    for (int r = lane; r < G; r += 32) {
                        int tok = r;
                        if (p.token_idx) {
                            const int v = p.token_idx[(int64_t)f * G + r];
                            if ((v < 0 || v >= p.n_in) && p.flags) atomicOr(p.flags, STOM_FLAG_BAD_INDEX);
                            tok = min(max(v, 0), p.n_in - 1);
                        }
                        bulk_load(dst + (uint32_t)r * ROW_BYTES, src + (int64_t)tok * p.st, ROW_BYTES, bar);
                    }
                    if (++slot == N) {
                        slot = 0;
                        ++round;
                    }
                }
            }
        }
        // nothing may still be landing in this block's shared memory when it exits: lane s looks after slot s and
        // waits for its latest fill.  On the regular path every fill has been consumed already and these waits
        // return at once.
        __syncwarp();
        if (lane < N) {
            const int32_t r = info[lane].round;
            if (r >= 0) mbar_wait(full_bar(lane, (uint32_t)r), ((uint32_t)r >> 1) & 1u, abort_flag + 1);
        }
        return;
    }

    // =================================================================== consumers
    if ((uint32_t)warp >= WA) return;
    int slot = warp;       // n_warps <= N
    uint32_t round = 0;    // fill number of `slot` that holds tile n
    for (uint32_t n = warp; n < my_count; n += WA) {
        // A parity wait cannot tell the fill it is waiting for from the fill two rounds back on the same barrier,
        // and the producer fills the slots of a group in whatever order they come free, so that older fill may
        // still be on its way when this warp gets here.  The producer publishes the fill number of a slot before it
        // starts the copy, and it starts that copy only after every earlier fill of the slot has been consumed.  So
        // the warp first waits (bounded) until the published number is its own: from then on the barrier has
        // completed exactly the earlier fills, and the parity wait that follows can only be answered by this one.
        bool ok = true;
        {
            unsigned long long t0 = 0;
            for (uint32_t spin = 0; *reinterpret_cast<volatile int32_t *>(&info[slot].round) != (int32_t)round; ++spin) {
                __nanosleep(32);
                if ((spin & 63u) == 63u) {
                    if (t0 == 0) t0 = global_ns();
                    if (*abort_flag || global_ns() - t0 > kWaitLimitNs) {
                        ok = false;
                        break;
                    }
                }
            }
            if (ok) ok = mbar_wait(full_bar(slot, round), (round >> 1) & 1u, abort_flag);
        }
        ok = __all_sync(0xffffffffu, ok && !*abort_flag);  // the whole warp stops together
        if (!ok) {
            if (lane == 0) {
                if (!*abort_flag && p.flags) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
                *abort_flag = 1;
            }
            break;
        }
        const unsigned char *tile = ring + (size_t)slot * p.slot_bytes + lane * LANE_BYTES;
        const int64_t bslot = info[slot].bslot;
        const int kind = info[slot].kind;
        const bool is_v = kind == 1;
        constexpr int md = MD;
        const bool want_sum = kind == 2 || (kind == 0 && p.n_kinds == 2);  // warp-uniform

        uint64_t sum2[C / 2];
#pragma unroll
        for (int j = 0; j < C / 2; ++j) sum2[j] = 0ull;  // (+0, +0)

        if (kind != 2) {
            // ---- pass 1: min / max of this lane's channels down the rows
            LaneRow<T, C> row;
            row.load(tile);
            uint32_t mnw[LaneRow<T, C>::W], mxw[LaneRow<T, C>::W];
#pragma unroll
            for (int j = 0; j < LaneRow<T, C>::W; ++j) mnw[j] = mxw[j] = row.w[j];
#pragma unroll 5
            for (int r = 1; r < G; ++r) {
                row.load(tile + r * ROW_BYTES);
#pragma unroll
                for (int j = 0; j < LaneRow<T, C>::W; ++j) {
                    mnw[j] = WordOps<T>::vmin(mnw[j], row.w[j]);
                    mxw[j] = WordOps<T>::vmax(mxw[j], row.w[j]);
                }
            }
            // ---- statistics of the lane's C channels
            float s[C], m[C], y[C];
            bool safe = true;
            {
                LaneRow<T, C> a, b;
#pragma unroll
                for (int j = 0; j < LaneRow<T, C>::W; ++j) {
                    a.w[j] = mnw[j];
                    b.w[j] = mxw[j];
                }
#pragma unroll
                for (int j = 0; j < C / 2; ++j) {
                    float mx0, mx1;
                    a.pair(j, m[2 * j], m[2 * j + 1]);
                    b.pair(j, mx0, mx1);
                    if (md != STOM_FP32) {  // warp-uniform
                        m[2 * j] = meta_round_down(m[2 * j], md);
                        m[2 * j + 1] = meta_round_down(m[2 * j + 1], md);
                    }
                    s[2 * j] = __fdiv_rn(__fsub_rn(mx0, m[2 * j]), kLevels);
                    s[2 * j + 1] = __fdiv_rn(__fsub_rn(mx1, m[2 * j + 1]), kLevels);
                    if (md != STOM_FP32) {
                        s[2 * j] = meta_round_up(s[2 * j], md);
                        s[2 * j + 1] = meta_round_up(s[2 * j + 1], md);
                    }
                }
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    safe &= (s[c] > 8.673617379884035e-19f) && (s[c] < 1.152921504606847e18f);  // (2^-60, 2^60)
                    y[c] = __frcp_rn(s[c]);
                }
            }
            store_meta<C>(is_v ? p.scale_v : p.scale_k, bslot * D + lane * C, md, s);
            store_meta<C>(is_v ? p.zero_v : p.zero_k, bslot * D + lane * C, md, m);
            safe = __all_sync(0xffffffffu, safe);

            unsigned char *out_lane = (is_v ? p.codes_v : p.codes_k) + bslot * (int64_t)code_bytes + lane * C * BITS / 8;

            // ---- pass 2: codes (and, for keys, the channel sums of the rows as a by-product)
            if (safe) {
                uint64_t m2[C / 2], ns2[C / 2], y2[C / 2], yl2[C / 2];
#pragma unroll
                for (int j = 0; j < C / 2; ++j) {
                    m2[j] = pack_f2(m[2 * j], m[2 * j + 1]);
                    ns2[j] = pack_f2(-s[2 * j], -s[2 * j + 1]);
                    y2[j] = pack_f2(y[2 * j], y[2 * j + 1]);
                    // what rn(1/s) leaves out: (1 - s*y) / s, the residual being exact in one FMA
                    yl2[j] = pack_f2(__fmul_rn(__fmaf_rn(-s[2 * j], y[2 * j], 1.0f), y[2 * j]),
                                     __fmul_rn(__fmaf_rn(-s[2 * j + 1], y[2 * j + 1], 1.0f), y[2 * j + 1]));
                }
                if (want_sum) code_rows<T, C, BITS, true>(tile, out_lane, G, lane, m2, ns2, y2, yl2, sum2);
                else code_rows<T, C, BITS, false>(tile, out_lane, G, lane, m2, ns2, y2, yl2, sum2);
            } else {
#pragma unroll 2
                for (int r = 0; r < G; ++r) {
                    row.load(tile + r * ROW_BYTES);
                    uint32_t cw = 0;
#pragma unroll
                    for (int j = 0; j < C / 2; ++j) {
                        float x0, x1;
                        row.pair(j, x0, x1);
                        if (want_sum) sum2[j] = add2(sum2[j], pack_f2(x0, x1));
                        cw |= code_slow(x0, m[2 * j], s[2 * j], kLevels) << (2 * BITS * j);
                        cw |= code_slow(x1, m[2 * j + 1], s[2 * j + 1], kLevels) << (2 * BITS * j + BITS);
                    }
                    store_codes<C, BITS>(out_lane + r * CODE_ROW, cw, lane);
                }
            }
            // the input slot is free again
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * slot);
        } else {
            // ---- pre-rotary keys: only their mean is wanted
            LaneRow<T, C> row;
#pragma unroll 5
            for (int r = 0; r < G; ++r) {
                row.load(tile + r * ROW_BYTES);
#pragma unroll
                for (int j = 0; j < C / 2; ++j) {
                    float x0, x1;
                    row.pair(j, x0, x1);
                    sum2[j] = add2(sum2[j], pack_f2(x0, x1));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * slot);
        }

        if (want_sum) {
            // ---- representative key: mean over the G tokens, and |k-bar_h|^2 over the head's d channels
            float kb[C];
            const float Gf = (float)G;
            float n2 = 0.0f;
#pragma unroll
            for (int j = 0; j < C / 2; ++j) {
                float a, b;
                unpack_f2(sum2[j], a, b);
                kb[2 * j] = __fdiv_rn(a, Gf);
                kb[2 * j + 1] = __fdiv_rn(b, Gf);
                if (md != STOM_FP32) {  // the norm below is the norm of the stored key
                    kb[2 * j] = meta_round_nearest(kb[2 * j], md);
                    kb[2 * j + 1] = meta_round_nearest(kb[2 * j + 1], md);
                }
            }
#pragma unroll
            for (int c = 0; c < C; ++c) n2 = fmaf(kb[c], kb[c], n2);
            store_meta<C>(p.rep_key, bslot * D + lane * C, md, kb);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
            if (lane == 0) p.rep_norm2[bslot] = n2;
        }
        slot += (int)WA;
        if (slot >= N) {
            slot -= N;
            ++round;
        }
    }
}

template <typename T, int C, int BITS, int MD>
static int32_t launch_quantize(QuantParams p, cudaStream_t stream) {
    int dev = 0, sms = 0, smem_max = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    const int G = p.g.G, D = 32 * C;
    const int tile_bytes = G * D * (int)sizeof(T);
    p.slot_bytes = (tile_bytes + 127) & ~127;
    // the ring takes all the shared memory there is; consumer warps never outnumber its slots
    int slots = (smem_max - kBarBytes) / p.slot_bytes;
    if (slots > kMaxSlots) slots = kMaxSlots;
    if (slots < 2) return STOM_ERR_SHAPE;
    p.n_slots = slots;
    p.n_warps = slots < kConsumerWarps ? slots : kConsumerWarps;
    const int fixed = kBarBytes;
    const size_t smem = (size_t)fixed + (size_t)slots * p.slot_bytes;
    e = cudaFuncSetAttribute(quantize_kernel<T, C, BITS, MD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    const unsigned grid = p.n_tiles < (uint32_t)sms ? p.n_tiles : (unsigned)sms;
    e = launch_after_producer(quantize_kernel<T, C, BITS, MD>, dim3(grid), dim3(kQuantThreads), smem, stream, p);
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    return finish_launch();
}

template <typename T, int C, int BITS>
static int32_t launch_for_meta(const QuantParams &p, cudaStream_t stream) {
    switch (p.g.meta_dtype) {
    case STOM_BF16: return launch_quantize<T, C, BITS, STOM_BF16>(p, stream);
    case STOM_FP16: return launch_quantize<T, C, BITS, STOM_FP16>(p, stream);
    default: return launch_quantize<T, C, BITS, STOM_FP32>(p, stream);
    }
}

template <typename T>
static int32_t launch_for_type(const QuantParams &p, int bits, cudaStream_t stream) {
    switch (p.g.d) {
    case 64: return bits == 4 ? launch_for_meta<T, 2, 4>(p, stream) : launch_for_meta<T, 2, 2>(p, stream);
    case 128: return bits == 4 ? launch_for_meta<T, 4, 4>(p, stream) : launch_for_meta<T, 4, 2>(p, stream);
    case 256: return bits == 4 ? launch_for_meta<T, 8, 4>(p, stream) : launch_for_meta<T, 8, 2>(p, stream);
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
    p.layer_begin = layer_begin; p.group_begin = group_begin; p.n_in = tokens_per_frame_in;
    p.flags = dev_flags;
    p.n_kinds = K_summary ? 3 : 2;
    p.contiguous = (!token_idx && stride_token == cfg->head_dim) ? 1 : 0;
    p.n_slots = 0; p.n_warps = 0; p.slot_bytes = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // one launch covers up to 2^30 tiles; longer frame ranges go out in slices
    const int64_t per_frame = (int64_t)layer_count * cfg->n_kv_heads * p.n_kinds;
    if (per_frame > (1 << 30)) return STOM_ERR_SHAPE;
    const int64_t max_frames = (1 << 30) / per_frame;
    const int eb = elem_bytes(dt);
    for (int64_t f0 = 0; f0 < group_count; f0 += max_frames) {
        QuantParams q = p;
        const int64_t nf = group_count - f0 < max_frames ? group_count - f0 : max_frames;
        const int64_t shift = f0 * stride_group * eb;
        q.K = static_cast<const uint8_t *>(K) + shift;
        q.V = static_cast<const uint8_t *>(V) + shift;
        if (K_summary) q.Ksum = static_cast<const uint8_t *>(K_summary) + shift;
        if (token_idx) q.token_idx = token_idx + f0 * cfg->group_tokens;
        q.group_begin = group_begin + (int32_t)f0;
        q.F = (int32_t)nf;
        q.n_tiles = (uint32_t)(per_frame * nf);
        switch (dt) {
        case STOM_BF16: rc = launch_for_type<__nv_bfloat16>(q, cfg->bits, s); break;
        case STOM_FP16: rc = launch_for_type<__half>(q, cfg->bits, s); break;
        default: rc = launch_for_type<float>(q, cfg->bits, s); break;
        }
        if (rc) return rc;
    }
    return STOM_OK;
}
