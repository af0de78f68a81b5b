// The specified steps of Causal Temporal Reduction (paper Sec. 3.3): the
// per-token temporal similarity s_t^(i), the static / dynamic split at tau_c,
// the proportional budget (k_s, k_d) and the saliency selection of the dynamic
// tokens.  The Merge of the static tokens is not here: the paper does not
// define it.
//
// similarity: HBM-bound streaming (every feature row is needed twice, as
//   "current" and as "previous").  A warp owns one token position over a run
//   of consecutive frames and keeps the previous frame's row and its squared
//   norm in registers, so a row is fetched from memory once (plus one row per
//   run); the row of the next frame is requested before the current one is
//   reduced.  Consecutive warps take consecutive positions of the same frames,
//   so the rows a block fetches are adjacent in memory.
// select: one block per frame.  N is a few hundred at most, so the top-k_d is
//   a rank count over the dynamic tokens in shared memory (a token is selected
//   if fewer than k_d dynamic tokens beat it; an equal saliency at a lower
//   index beats it), between two ordered compactions -- exact, and already in
//   ascending order.
#include "stom_internal.cuh"

#include "stom_ctr.h"

namespace stom {

constexpr int kSimWarps = 8;
constexpr int kSimRun = 32;  // frames one warp walks; one extra row is read per run

struct SimParams {
    const void *F, *prev;
    int64_t sf, st;  // element strides: frame, token
    float *sim;
    int32_t T, N, D, n_runs;
};

__device__ __forceinline__ uint64_t pair_f2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void split_f2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// T: element type; NP: 16-byte vectors of a row per lane
// Blocks of wide rows are half as large: a thread then holds so many registers that whole blocks of 8 warps would
// leave a third of the register file idle.
template <int NP>
__host__ __device__ constexpr int sim_warps() { return NP > 8 ? kSimWarps / 2 : kSimWarps; }

template <typename T, int NP>
__global__ void __launch_bounds__(sim_warps<NP>() * 32) ctr_similarity_kernel(const SimParams p) {
    constexpr int EPV = 16 / (int)sizeof(T);  // elements per vector
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t w = (int64_t)blockIdx.x * sim_warps<NP>() + warp;
    if (w >= (int64_t)p.n_runs * p.N) return;
    const int run = (int)(w / p.N), i = (int)(w - (int64_t)run * p.N);
    const int f0 = run * kSimRun, f1 = min(f0 + kSimRun, p.T);
    const T *base = static_cast<const T *>(p.F) + (int64_t)i * p.st;

    auto load_row = [&](const T *row, uint4 (&v)[NP]) {
#pragma unroll
        for (int q = 0; q < NP; ++q) {
            const int e = (q * 32 + lane) * EPV;
            v[q] = e < p.D ? __ldg(reinterpret_cast<const uint4 *>(row + e)) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    // sum over the lane's elements of a*b and of a*a.  Rows of up to 4 KB: two channels per instruction (f32x2),
    // which also keeps the kernel at three blocks per SM; wider rows measured faster with scalar accumulation.
    auto dots = [&](const uint4 (&a)[NP], const uint4 (&b)[NP], float &ab, float &aa) {
        if constexpr (NP > 8) {
            float s_ab = 0.0f, s_aa = 0.0f;
#pragma unroll
            for (int q = 0; q < NP; ++q) {
                const uint32_t aw[4] = {a[q].x, a[q].y, a[q].z, a[q].w}, bw[4] = {b[q].x, b[q].y, b[q].z, b[q].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (sizeof(T) == 4) {
                        s_ab = fmaf(__uint_as_float(aw[j]), __uint_as_float(bw[j]), s_ab);
                        s_aa = fmaf(__uint_as_float(aw[j]), __uint_as_float(aw[j]), s_aa);
                    } else {
                        float a0, a1, b0, b1;
                        unpack2<T>(aw[j], a0, a1);
                        unpack2<T>(bw[j], b0, b1);
                        s_ab = fmaf(a0, b0, s_ab);
                        s_ab = fmaf(a1, b1, s_ab);
                        s_aa = fmaf(a0, a0, s_aa);
                        s_aa = fmaf(a1, a1, s_aa);
                    }
                }
            }
            ab = s_ab;
            aa = s_aa;
            return;
        }
        uint64_t acc_ab = 0ull, acc_aa = 0ull;  // (+0, +0)
#pragma unroll
        for (int q = 0; q < NP; ++q) {
            const uint32_t aw[4] = {a[q].x, a[q].y, a[q].z, a[q].w}, bw[4] = {b[q].x, b[q].y, b[q].z, b[q].w};
            if constexpr (sizeof(T) == 4) {
#pragma unroll
                for (int j = 0; j < 4; j += 2) {
                    const uint64_t a2 = pair_f2(__uint_as_float(aw[j]), __uint_as_float(aw[j + 1]));
                    const uint64_t b2 = pair_f2(__uint_as_float(bw[j]), __uint_as_float(bw[j + 1]));
                    acc_ab = fma_f2(a2, b2, acc_ab);
                    acc_aa = fma_f2(a2, a2, acc_aa);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float a0, a1, b0, b1;
                    unpack2<T>(aw[j], a0, a1);
                    unpack2<T>(bw[j], b0, b1);
                    const uint64_t a2 = pair_f2(a0, a1), b2 = pair_f2(b0, b1);
                    acc_ab = fma_f2(a2, b2, acc_ab);
                    acc_aa = fma_f2(a2, a2, acc_aa);
                }
            }
        }
        float lo, hi;
        split_f2(acc_ab, lo, hi);
        ab = lo + hi;
        split_f2(acc_aa, lo, hi);
        aa = lo + hi;
    };
    auto warp_sum = [](float v) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        return v;
    };

    uint4 prv[NP], cur[NP];
    bool have_prev = true;
    if (f0 > 0) {
        load_row(base + (int64_t)(f0 - 1) * p.sf, prv);
    } else if (p.prev) {
        load_row(static_cast<const T *>(p.prev) + (int64_t)i * p.st, prv);
    } else {
        have_prev = false;  // the first frame of a stream
#pragma unroll
        for (int q = 0; q < NP; ++q) prv[q] = make_uint4(0u, 0u, 0u, 0u);
    }
    load_row(base + (int64_t)f0 * p.sf, cur);
    float n_prv, unused;
    dots(prv, prv, unused, n_prv);
    n_prv = warp_sum(n_prv);
    for (int f = f0; f < f1; ++f) {
        uint4 nxt[NP];
        if (f + 1 < f1) load_row(base + (int64_t)(f + 1) * p.sf, nxt);
        float d, n_cur;
        dots(cur, prv, d, n_cur);
        d = warp_sum(d);
        n_cur = warp_sum(n_cur);
        if (lane == 0) {
            const float den = fmaxf(sqrtf(n_cur), 1e-12f) * fmaxf(sqrtf(n_prv), 1e-12f);
            p.sim[(int64_t)f * p.N + i] = have_prev ? d / den : -INFINITY;
        }
        have_prev = true;
        n_prv = n_cur;
#pragma unroll
        for (int q = 0; q < NP; ++q) {
            prv[q] = cur[q];
            if (f + 1 < f1) cur[q] = nxt[q];
        }
    }
}

constexpr int kSelThreads = 256;
constexpr int kSelMaxTokens = 1024;

struct SelParams {
    const float *sim, *alpha;
    int32_t *k_s, *k_d, *static_idx, *dyn_idx;
    int32_t N, G;
    float tau;
};

// Ordered split of the block's items [0, n) by flag(i): calls put(i, rank among the flagged, flagged?) for every
// item, ranks ascending in i (for an item that is not flagged the rank counts the flagged ones before it), and
// returns how many are flagged.  All threads of the block call it.
template <typename Flag, typename Put>
__device__ __forceinline__ int ordered_split(int n, uint32_t *warp_tot, Flag flag, Put put) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int seen = 0;
    for (int b0 = 0; b0 < n; b0 += kSelThreads) {
        const int i = b0 + tid;
        const bool f = i < n && flag(i);
        const uint32_t m = __ballot_sync(0xffffffffu, f);
        if (lane == 0) warp_tot[warp] = __popc(m);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int wq = 0; wq < kSelThreads / 32; ++wq) {
            const int c = (int)warp_tot[wq];
            before += wq < warp ? c : 0;
            total += c;
        }
        if (i < n) put(i, seen + before + __popc(m & ((1u << lane) - 1u)), f);
        seen += total;
        __syncthreads();  // warp_tot is rewritten by the next trip
    }
    return seen;
}

__global__ void __launch_bounds__(kSelThreads) ctr_select_kernel(const SelParams p) {
    __shared__ float d_alpha[kSelMaxTokens];    // saliency of the dynamic tokens, in ascending token order
    __shared__ int16_t d_token[kSelMaxTokens];  // their token indices
    __shared__ uint8_t d_sel[kSelMaxTokens];
    __shared__ uint32_t warp_tot[kSelThreads / 32];
    const int t = blockIdx.x, N = p.N, tid = threadIdx.x;
    const float *sim = p.sim + (int64_t)t * N, *alpha = p.alpha + (int64_t)t * N;
    int32_t *s_out = p.static_idx + (int64_t)t * N, *d_out = p.dyn_idx + (int64_t)t * p.G;
    // S_t goes out in ascending order; D_t is listed in shared memory, ascending too (a token's place among the
    // dynamic ones is its index minus the static tokens before it)
    const int n_s = ordered_split(
        N, warp_tot, [&](int i) { return sim[i] > p.tau; },
        [&](int i, int rank, bool is_static) {
            if (is_static) {
                s_out[rank] = i;
            } else {
                d_alpha[i - rank] = alpha[i];
                d_token[i - rank] = (int16_t)i;
            }
        });
    for (int j = n_s + tid; j < N; j += kSelThreads) s_out[j] = -1;
    const int n_d = N - n_s;
    const int k_s = (int)(((int64_t)p.G * n_s) / N), k_d = p.G - k_s;
    if (tid == 0) {
        p.k_s[t] = k_s;
        p.k_d[t] = k_d;
    }
    __syncthreads();
    // a dynamic token is selected if fewer than k_d dynamic tokens come before it in (saliency descending, index
    // ascending) order: a rank count over the dynamic list only
    for (int r = tid; r < n_d; r += kSelThreads) {
        const float ai = d_alpha[r];
        int rank = 0;
        for (int j = 0; j < n_d; ++j) rank += d_alpha[j] > ai || (d_alpha[j] == ai && j < r);
        d_sel[r] = rank < k_d;
    }
    __syncthreads();
    const int n_sel = ordered_split(
        n_d, warp_tot, [&](int r) { return d_sel[r] != 0; },
        [&](int r, int rank, bool sel) {
            if (sel) d_out[rank] = d_token[r];
        });
    for (int j = n_sel + tid; j < p.G; j += kSelThreads) d_out[j] = -1;
}

template <typename T, int NP>
static void launch_similarity_np(const SimParams &p, cudaStream_t s) {
    constexpr int W = sim_warps<NP>();
    const int64_t warps = (int64_t)p.n_runs * p.N;
    ctr_similarity_kernel<T, NP><<<(unsigned)((warps + W - 1) / W), W * 32, 0, s>>>(p);
}

template <typename T>
static void launch_similarity(const SimParams &p, int np, cudaStream_t s) {
    switch (np) {
    case 1: launch_similarity_np<T, 1>(p, s); break;
    case 2: launch_similarity_np<T, 2>(p, s); break;
    case 3: launch_similarity_np<T, 3>(p, s); break;
    case 4: launch_similarity_np<T, 4>(p, s); break;
    case 5: launch_similarity_np<T, 5>(p, s); break;
    case 6: launch_similarity_np<T, 6>(p, s); break;
    case 7: launch_similarity_np<T, 7>(p, s); break;
    case 8: launch_similarity_np<T, 8>(p, s); break;
    case 9: case 10: launch_similarity_np<T, 10>(p, s); break;
    case 11: case 12: launch_similarity_np<T, 12>(p, s); break;
    case 13: case 14: launch_similarity_np<T, 14>(p, s); break;
    default: launch_similarity_np<T, 16>(p, s); break;  // rows of up to 8 KB
    }
}

}  // namespace stom

using namespace stom;

extern "C" int32_t stom_ctr_similarity(const void *F, const void *prev, int32_t dtype, int32_t T, int32_t N, int32_t D,
                                       int64_t stride_frame, int64_t stride_token, float *sim, void *stream) {
    if (!F || !sim || T < 0 || N < 1 || D < 1) return STOM_ERR_INVALID_ARG;
    if (dtype != STOM_BF16 && dtype != STOM_FP16 && dtype != STOM_FP32) return STOM_ERR_UNSUPPORTED;
    const int epv = 16 / elem_bytes(dtype);
    if (D % epv || D * elem_bytes(dtype) > 16 * 512 || N > (1 << 20)) return STOM_ERR_SHAPE;
    if (stride_token < D || stride_frame < 0) return STOM_ERR_INVALID_ARG;
    if (!aligned16(F) || (prev && !aligned16(prev)) || (reinterpret_cast<uintptr_t>(sim) & 3u)) return STOM_ERR_ALIGNMENT;
    if (!stride_ok(stride_frame, dtype) || !stride_ok(stride_token, dtype)) return STOM_ERR_ALIGNMENT;
    if (T == 0) return STOM_OK;
    SimParams p;
    p.F = F; p.prev = prev; p.sf = stride_frame; p.st = stride_token; p.sim = sim;
    p.T = T; p.N = N; p.D = D;
    p.n_runs = (T + kSimRun - 1) / kSimRun;
    if ((int64_t)p.n_runs * N > 0x7fffffffLL) return STOM_ERR_SHAPE;
    const int np = (D * elem_bytes(dtype) + 511) / 512;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (dtype) {
    case STOM_BF16: launch_similarity<__nv_bfloat16>(p, np, s); break;
    case STOM_FP16: launch_similarity<__half>(p, np, s); break;
    default: launch_similarity<float>(p, np, s); break;
    }
    return finish_launch();
}

extern "C" int32_t stom_ctr_select(const float *sim, const float *alpha, int32_t T, int32_t N, int32_t G, float tau_c,
                                   int32_t *k_s, int32_t *k_d, int32_t *static_idx, int32_t *dyn_idx, void *stream) {
    if (!sim || !alpha || !k_s || !k_d || !static_idx || !dyn_idx || T < 0 || N < 1 || G < 1) return STOM_ERR_INVALID_ARG;
    if (G > N || N > kSelMaxTokens) return STOM_ERR_SHAPE;
    const void *ptrs[6] = {sim, alpha, k_s, k_d, static_idx, dyn_idx};
    for (const void *q : ptrs)
        if (reinterpret_cast<uintptr_t>(q) & 3u) return STOM_ERR_ALIGNMENT;
    if (T == 0) return STOM_OK;
    SelParams p{sim, alpha, k_s, k_d, static_idx, dyn_idx, N, G, tau_c};
    ctr_select_kernel<<<(unsigned)T, kSelThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return finish_launch();
}

extern "C" int32_t stom_ctr_reduce(const void *F, const void *prev, int32_t dtype, int32_t T, int32_t N, int32_t D,
                                   int64_t stride_frame, int64_t stride_token, const float *alpha, int32_t G,
                                   float tau_c, float *sim, int32_t *k_s, int32_t *k_d, int32_t *static_idx,
                                   int32_t *dyn_idx, void *stream) {
    // both argument lists are checked before the first launch
    if (!alpha || !k_s || !k_d || !static_idx || !dyn_idx || G < 1 || N < 1) return STOM_ERR_INVALID_ARG;
    if (G > N || N > kSelMaxTokens) return STOM_ERR_SHAPE;
    const void *ptrs[5] = {alpha, k_s, k_d, static_idx, dyn_idx};
    for (const void *q : ptrs)
        if (reinterpret_cast<uintptr_t>(q) & 3u) return STOM_ERR_ALIGNMENT;
    int32_t rc = stom_ctr_similarity(F, prev, dtype, T, N, D, stride_frame, stride_token, sim, stream);
    if (rc) return rc;
    return stom_ctr_select(sim, alpha, T, N, G, tau_c, k_s, k_d, static_idx, dyn_idx, stream);
}
