// Device code of A3 (top-K group selection, ascending output; paper Sec. 3.4 TopK, appendix "Question-guided
// single-pass retrieval"), shared by the stand-alone kernel and by the fused retrieval kernel.
#pragma once

#include "stom_internal.cuh"

namespace stom {

constexpr int kTopkBlock = 1024;          // threads of the stand-alone kernel
constexpr int kTopkRegKeys = 8;           // keys a thread holds in registers
constexpr int kTopkSmemKeys = 48 * 1024;  // rows up to this many scores are staged in shared memory

enum { kKeysGlobal = 0, kKeysShared = 1, kKeysRegs = 2 };

__device__ __forceinline__ uint32_t score_key(float f) {
    f += 0.0f;  // -0 -> +0, so that equal scores have equal keys
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct TopkParams {
    const float *scores;
    int64_t row_stride;
    int32_t n, k;
    int32_t *idx_out;
    float *score_out;
    int32_t *n_sel_out;
};

// Scratch of one block-wide selection.
struct TopkSmem {
    uint32_t hist[256];
    uint32_t s_prefix, s_need, s_done;
    uint32_t warp_gt[32], warp_eq[32];
};

// Top-K of one row by the NT threads of a block (all of them must call).  sc: the row's n scores; idx_out [k],
// score_out [k] (nullable), n_sel_out (nullable, one int); skeys: n words of shared memory in mode kKeysShared.
// Scores are read through L2 only (ld.cg), so the row may have been written by other blocks of the same launch
// once their writes are fenced.
template <int NT, int MODE>
__device__ __forceinline__ void block_topk(const float *sc, int n, int k, int32_t *idx_out, float *score_out,
                                           int32_t *n_sel_out, uint32_t *skeys, TopkSmem &sm) {
    uint32_t(&hist)[256] = sm.hist;
    uint32_t &s_prefix = sm.s_prefix, &s_need = sm.s_need, &s_done = sm.s_done;
    uint32_t(&warp_gt)[32] = sm.warp_gt, (&warp_eq)[32] = sm.warp_eq;
    constexpr int kTopkThreads = NT;
    const int tid = threadIdx.x;
    const int ksel = min(k, n);

    if (tid == 0 && n_sel_out) *n_sel_out = ksel;
    for (int j = ksel + tid; j < k; j += kTopkThreads) {  // unused slots
        idx_out[j] = -1;
        if (score_out) score_out[j] = 0.0f;
    }
    if (ksel == 0) return;

    // thread `tid` owns the contiguous index range [lo, hi)
    const int per = MODE == kKeysRegs ? kTopkRegKeys : (n + kTopkThreads - 1) / kTopkThreads;
    const int lo = min(tid * per, n), hi = min(lo + per, n);

    uint32_t rk[kTopkRegKeys];  // kKeysRegs: the thread's keys; slots past hi hold 0 and are never counted
    if constexpr (MODE == kKeysRegs) {
        const bool vec = ((reinterpret_cast<uintptr_t>(sc) & 15u) == 0) && lo + kTopkRegKeys <= n;
        if (vec) {
#pragma unroll
            for (int e = 0; e < kTopkRegKeys; e += 4) {
                const float4 v = __ldcg(reinterpret_cast<const float4 *>(sc + lo + e));
                rk[e] = score_key(v.x); rk[e + 1] = score_key(v.y); rk[e + 2] = score_key(v.z); rk[e + 3] = score_key(v.w);
            }
        } else {
#pragma unroll
            for (int e = 0; e < kTopkRegKeys; ++e) rk[e] = lo + e < hi ? score_key(__ldcg(sc + lo + e)) : 0u;
        }
    } else if constexpr (MODE == kKeysShared) {
        for (int i = tid; i < n; i += kTopkThreads) skeys[i] = score_key(__ldcg(sc + i));
        __syncthreads();
    }
    // visits the thread's keys in index order: f(index, key)
    auto for_my_keys = [&](auto &&f) {
        if constexpr (MODE == kKeysRegs) {
#pragma unroll
            for (int e = 0; e < kTopkRegKeys; ++e)
                if (lo + e < hi) f(lo + e, rk[e]);
        } else {
            for (int i = lo; i < hi; ++i) {
                if constexpr (MODE == kKeysShared) f(i, skeys[i]);
                else f(i, score_key(__ldcg(sc + i)));
            }
        }
    };

    // ---- radix select of the ksel-th largest key: up to 4 passes of 8 bits.  The bin in which the running count from
    //      the top reaches `need` is found by one warp: a lane owns 8 bins, suffix sums go round by shuffle.  The
    //      passes stop as soon as that bin has exactly as many keys as are still needed: all of them are taken, so
    //      their lower bits no longer matter (with well-spread scores that is after two passes).
    uint32_t prefix = 0, mask = 0, need = (uint32_t)ksel;
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for_my_keys([&](int, uint32_t key) {
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        });
        __syncthreads();
        if (tid < 32) {
            uint32_t c[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c[j] = hist[tid * 8 + j];
                tot += c[j];
            }
            uint32_t suf = tot;  // becomes the count in this lane's bins and all higher ones
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_down_sync(0xffffffffu, suf, o);
                if (tid + o < 32) suf += v;
            }
            const uint32_t above = suf - tot;
            if (above < need && need <= suf) {  // exactly one lane: 1 <= need <= number of candidates
                uint32_t left = need - above;
                int j = 7;
                for (; j > 0; --j) {
                    if (c[j] >= left) break;
                    left -= c[j];
                }
                s_prefix = prefix | ((uint32_t)(tid * 8 + j) << shift);
                s_need = left;
                s_done = c[j] == left;
            }
        }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
        mask |= 255u << shift;
        if (s_done) break;  // block-uniform
    }
    // keys whose bits under `mask` exceed `prefix` are taken; of those that equal it, the first `need` in index order
    // (after all four passes `prefix` is the exact key of the ksel-th largest)

    // ---- ordered compaction over the threads' contiguous ranges
    uint32_t gt = 0, eq = 0;
    for_my_keys([&](int, uint32_t key) {
        gt += (key & mask) > prefix;
        eq += (key & mask) == prefix;
    });
    // exclusive prefix sums of (gt, eq) over threads: warp scan, then scan of warp totals
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t igt = gt, ieq = eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t a = __shfl_up_sync(0xffffffffu, igt, o);
        const uint32_t b = __shfl_up_sync(0xffffffffu, ieq, o);
        if (lane >= o) {
            igt += a;
            ieq += b;
        }
    }
    if (lane == 31) {
        warp_gt[warp] = igt;
        warp_eq[warp] = ieq;
    }
    __syncthreads();
    if (warp == 0) {
        uint32_t a = lane < NT / 32 ? warp_gt[lane] : 0u, b = lane < NT / 32 ? warp_eq[lane] : 0u;
        uint32_t ia = a, ib = b;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t x = __shfl_up_sync(0xffffffffu, ia, o);
            const uint32_t y = __shfl_up_sync(0xffffffffu, ib, o);
            if (lane >= o) {
                ia += x;
                ib += y;
            }
        }
        warp_gt[lane] = ia - a;  // exclusive
        warp_eq[lane] = ib - b;
    }
    __syncthreads();
    uint32_t gt_before = warp_gt[warp] + igt - gt;
    uint32_t eq_before = warp_eq[warp] + ieq - eq;
    for_my_keys([&](int i, uint32_t key) {
        const bool take = (key & mask) > prefix || ((key & mask) == prefix && eq_before < need);
        if (take) {
            const uint32_t pos = gt_before + min(eq_before, need);
            idx_out[pos] = i;
            if (score_out) score_out[pos] = __ldcg(sc + i);
        }
        gt_before += (key & mask) > prefix;
        eq_before += (key & mask) == prefix;
    });
}


template <int MODE>
__global__ void __launch_bounds__(kTopkBlock) topk_kernel(const TopkParams p) {
    extern __shared__ __align__(16) uint32_t skeys[];  // kKeysShared: n keys
    __shared__ TopkSmem sm;
    const int row = blockIdx.x;
    block_topk<kTopkBlock, MODE>(p.scores + (int64_t)row * p.row_stride, p.n, p.k, p.idx_out + (int64_t)row * p.k,
                                 p.score_out ? p.score_out + (int64_t)row * p.k : nullptr,
                                 p.n_sel_out ? p.n_sel_out + row : nullptr, skeys, sm);
}

}  // namespace stom
