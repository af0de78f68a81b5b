// A3: top-K group selection (paper Sec. 3.4, R = TopK{sim(q, k-bar_i)};
// appendix: K = min(ceil(B/G), T/G) and the selected indices stay in sorted,
// i.e. chronological, order).
//
// One thread block per row.  Scores become order-preserving 32-bit keys; a
// most-significant-digit radix select (4 passes of 8 bits, shared-memory
// histogram, the crossing bin found by one warp with shuffles) finds the K-th
// largest key exactly; a block-wide ordered compaction then emits, in
// ascending index order, every element above that key plus the first `need`
// elements equal to it -- so equal scores resolve to the lower index and the
// output needs no sort.  No thread ever waits on another block.
//
// A thread owns a contiguous run of the row.  Rows of up to 8 x 1024 scores
// (every workload of the paper's geometry: one score per stored frame) keep
// their keys in registers; longer rows stage them in shared memory, and rows
// beyond that re-read the scores from global memory in every pass.
#include "stom_internal.cuh"

namespace stom {

constexpr int kTopkThreads = 1024;
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

template <int MODE>
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const TopkParams p) {
    extern __shared__ __align__(16) uint32_t skeys[];  // kKeysShared: n keys
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_need;
    __shared__ uint32_t warp_gt[32], warp_eq[32];

    const int row = blockIdx.x, tid = threadIdx.x, n = p.n;
    const float *sc = p.scores + (int64_t)row * p.row_stride;
    const int ksel = min(p.k, n);
    int32_t *idx_out = p.idx_out + (int64_t)row * p.k;
    float *score_out = p.score_out ? p.score_out + (int64_t)row * p.k : nullptr;

    if (tid == 0 && p.n_sel_out) p.n_sel_out[row] = ksel;
    for (int j = ksel + tid; j < p.k; j += kTopkThreads) {  // unused slots
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
                const float4 v = __ldg(reinterpret_cast<const float4 *>(sc + lo + e));
                rk[e] = score_key(v.x); rk[e + 1] = score_key(v.y); rk[e + 2] = score_key(v.z); rk[e + 3] = score_key(v.w);
            }
        } else {
#pragma unroll
            for (int e = 0; e < kTopkRegKeys; ++e) rk[e] = lo + e < hi ? score_key(__ldg(sc + lo + e)) : 0u;
        }
    } else if constexpr (MODE == kKeysShared) {
        for (int i = tid; i < n; i += kTopkThreads) skeys[i] = score_key(sc[i]);
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
                else f(i, score_key(__ldg(sc + i)));
            }
        }
    };

    // ---- radix select of the ksel-th largest key: 4 passes of 8 bits.  The bin in which the running count from the
    //      top reaches `need` is found by one warp: a lane owns 8 bins, suffix sums go round by shuffle.
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
            }
        }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
        mask |= 255u << shift;
    }
    const uint32_t kth = prefix;  // exact key of the ksel-th largest; `need` of the elements equal to it are taken

    // ---- ordered compaction over the threads' contiguous ranges
    uint32_t gt = 0, eq = 0;
    for_my_keys([&](int, uint32_t key) {
        gt += key > kth;
        eq += key == kth;
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
        uint32_t a = warp_gt[lane], b = warp_eq[lane];
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
        const bool take = key > kth || (key == kth && eq_before < need);
        if (take) {
            const uint32_t pos = gt_before + min(eq_before, need);
            idx_out[pos] = i;
            if (score_out) score_out[pos] = sc[i];
        }
        gt_before += key > kth;
        eq_before += key == kth;
    });
}

}  // namespace stom

using namespace stom;

extern "C" int32_t stom_oqm_topk(const float *scores, int32_t rows, int32_t n, int64_t row_stride, int32_t k,
                                 int32_t *idx_out, float *score_out, int32_t *n_sel_out, void *stream) {
    if (!scores || !idx_out || rows < 0 || n < 0 || k < 1 || row_stride < n) return STOM_ERR_INVALID_ARG;
    if (n > (1 << 24)) return STOM_ERR_SHAPE;
    if (rows == 0) return STOM_OK;
    TopkParams p{scores, row_stride, n, k, idx_out, score_out, n_sel_out};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n <= kTopkRegKeys * kTopkThreads) {
        topk_kernel<kKeysRegs><<<rows, kTopkThreads, 0, s>>>(p);
    } else if (n <= kTopkSmemKeys) {
        const size_t smem = (size_t)n * sizeof(uint32_t);
        if (smem > 40 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(topk_kernel<kKeysShared>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 kTopkSmemKeys * (int)sizeof(uint32_t));
            if (e != cudaSuccess) {
                set_last_cuda_error(e);
                return STOM_ERR_CUDA;
            }
        }
        topk_kernel<kKeysShared><<<rows, kTopkThreads, smem, s>>>(p);
    } else {
        topk_kernel<kKeysGlobal><<<rows, kTopkThreads, 0, s>>>(p);
    }
    return finish_launch();
}
