// Device code of A2 (question embedding and cosine scores over the representative keys; paper appendix
// "Question-guided single-pass retrieval", Sec. 3.4 sim(q, k-bar_i)), shared by the stand-alone scoring kernels and
// by the fused retrieval kernel.
#pragma once

#include "stom_internal.cuh"

namespace stom {

struct ScoreParams {
    const void *Q;
    int64_t ql, qh, qt;  // element strides of Q: layer, head, token
    const void *rep_key;  // elements of g.meta_dtype
    const float *rep_norm2;
    float *qemb;    // workspace: [layer_count][H][d]
    float *qnorm2;  // workspace: [layer_count][H]
    float *scores;
    BankGeom g;
    int32_t layer_begin, layer_count, n_groups, T_q, rep, per_head, groups_per_block;
};

constexpr int kEmbedThreads = 256;

// Question embedding of one (layer, kv head): mean over the rep query heads of the GQA block and over the T_q
// question tokens.  grid (H, layer_count), kEmbedThreads threads.  The rows (rep * T_q of them) are dealt to
// RG = kEmbedThreads / (d/8) row groups; a thread adds up 8 adjacent channels (16-byte loads) of its group's rows,
// up to 16 rows in flight at once -- the kernel is a few memory round trips and nothing else -- and shared memory
// combines the groups.
template <typename T>
__global__ void __launch_bounds__(kEmbedThreads) query_embed_kernel(const ScoreParams p) {
    __shared__ __align__(16) float part[kEmbedThreads / 8][256 + 4];  // [row group <= 32][channel <= 256]
    __shared__ float red[kEmbedThreads / 32];
    grid_launch_dependents();  // the scoring kernel behind this one may be scheduled; it waits before it reads
    const int h = blockIdx.x, li = blockIdx.y, d = p.g.d;
    const int lanes_per_row = d >> 3;                 // threads across one row (8 channels each): 8, 16 or 32
    const int RG = kEmbedThreads / lanes_per_row;     // row groups: 32, 16 or 8
    const int cq = threadIdx.x % lanes_per_row, rg = threadIdx.x / lanes_per_row;
    const int rows = p.rep * p.T_q;
    const T *q = reinterpret_cast<const T *>(p.Q) + (int64_t)li * p.ql + (int64_t)h * p.rep * p.qh + cq * 8;
    float acc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = 0.0f;
    constexpr int kRowBatch = sizeof(T) == 4 ? 8 : 16;
    constexpr int W = 8 * (int)sizeof(T) / 4;  // 32-bit words of a thread's 8 channels
    // (hr, j): query head inside the block and token of the thread's current row, stepped without a division
    int hr = rg / p.T_q, j = rg - hr * p.T_q;
    for (int r0 = rg; r0 < rows; r0 += RG * kRowBatch) {
        uint32_t x[kRowBatch][W];
#pragma unroll
        for (int b = 0; b < kRowBatch; ++b) {
#pragma unroll
            for (int i = 0; i < W; ++i) x[b][i] = 0u;  // +0.0 in every format
            if (r0 + b * RG < rows) {
                const uint4 *src = reinterpret_cast<const uint4 *>(q + (int64_t)hr * p.qh + (int64_t)j * p.qt);
#pragma unroll
                for (int i = 0; i < W / 4; ++i) {
                    const uint4 v = __ldg(src + i);
                    x[b][4 * i] = v.x; x[b][4 * i + 1] = v.y; x[b][4 * i + 2] = v.z; x[b][4 * i + 3] = v.w;
                }
            }
            j += RG;
            while (j >= p.T_q) {
                j -= p.T_q;
                ++hr;
            }
        }
#pragma unroll
        for (int b = 0; b < kRowBatch; ++b) {
            if constexpr (sizeof(T) == 4) {
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[c] += __uint_as_float(x[b][c]);
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    float lo, hi;
                    unpack2<T>(x[b][c], lo, hi);
                    acc[2 * c] += lo;
                    acc[2 * c + 1] += hi;
                }
            }
        }
    }
    float4 *mine = reinterpret_cast<float4 *>(&part[rg][cq * 8]);
    mine[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    mine[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    __syncthreads();
    float sq = 0.0f;
    if (threadIdx.x < d) {
        const int c = threadIdx.x;
        float a = 0.0f;
        for (int g = 0; g < RG; ++g) a += part[g][c];
        const float v = a / (float)rows;
        p.qemb[((int64_t)li * p.g.H + h) * d + c] = v;
        sq = v * v;
    }
    // |q_h|^2 by block reduction
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.0f;
        for (int w = 0; w < kEmbedThreads / 32; ++w) tot += red[w];
        p.qnorm2[(int64_t)li * p.g.H + h] = tot;
    }
}

constexpr int kScoreWarps = 8;

// One warp, a strided share of the block's groups [t_begin, t_end) of one layer, kGroupsPerWarp at a time.  The
// loads of the next batch are issued before the current batch is reduced, so a warp always has 2 batches of k-bar
// vectors in flight.  V4: the flattened k-bar has H*d = 128 * V4 channels; KT: the type it is stored in.  A lane
// covers NV 16-byte vectors of each k-bar: vector i of a lane holds channels [(lane + 32 i) * E, ... + E).
template <int V4, typename KT>
__device__ __forceinline__ void score_groups_per_layer(const ScoreParams &p, const float *sq, const float *qn, int li,
                                                       int t_begin, int t_end, int warp, int lane) {
    constexpr int E = 16 / (int)sizeof(KT);  // channels per 16-byte vector
    constexpr int NV = V4 * 4 / E;           // vectors of one k-bar per lane
    static_assert(NV >= 1 && NV * E == V4 * 4, "k-bar must fill whole 16-byte vectors across the warp");
    // groups a warp scores together (register budget: about 8 vectors per batch)
    constexpr int kGroupsPerWarp = sizeof(KT) == 4 ? (V4 >= 8 ? 1 : 2) : (NV >= 4 ? 2 : 4);
    const int H = p.g.H, d = p.g.d, l = p.layer_begin + li;
    float q[NV][E];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
#pragma unroll
        for (int e = 0; e < E; e += 4) {
            const float4 v = reinterpret_cast<const float4 *>(sq)[((lane + 32 * i) * E + e) >> 2];
            q[i][e] = v.x; q[i][e + 1] = v.y; q[i][e + 2] = v.z; q[i][e + 3] = v.w;
        }
    }
    float qq = lane < H ? qn[lane] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) qq += __shfl_xor_sync(0xffffffffu, qq, o);
    const float qnorm = fmaxf(sqrtf(qq), 1e-12f);

    auto load = [&](int t0, uint4 (&kv)[kGroupsPerWarp][NV], float (&kn)[kGroupsPerWarp]) {
#pragma unroll
        for (int u = 0; u < kGroupsPerWarp; ++u) {
            const int t = min(t0 + u, t_end - 1);  // a batch that sticks out re-reads the last group; dropped at the store
            const int64_t slot = bank_slot(p.g, l, t, 0);
            const uint4 *kb = reinterpret_cast<const uint4 *>(static_cast<const KT *>(p.rep_key) + slot * d);
#pragma unroll
            for (int i = 0; i < NV; ++i) kv[u][i] = __ldg(kb + lane + 32 * i);
            kn[u] = lane < H ? __ldg(p.rep_norm2 + slot + lane) : 0.0f;
        }
    };
    const int step = kScoreWarps * kGroupsPerWarp;
    int t0 = t_begin + warp * kGroupsPerWarp;
    if (t0 >= t_end) return;
    uint4 cur[kGroupsPerWarp][NV], nxt[kGroupsPerWarp][NV];
    float kn_cur[kGroupsPerWarp], kn_nxt[kGroupsPerWarp];
    load(t0, cur, kn_cur);
    for (; t0 < t_end; t0 += step) {
        const bool more = t0 + step < t_end;
        if (more) load(t0 + step, nxt, kn_nxt);
        float dot[kGroupsPerWarp];
#pragma unroll
        for (int u = 0; u < kGroupsPerWarp; ++u) {
            float a = 0.0f;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t w[4] = {cur[u][i].x, cur[u][i].y, cur[u][i].z, cur[u][i].w};
                if constexpr (sizeof(KT) == 4) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) a = fmaf(__uint_as_float(w[e]), q[i][e], a);
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float lo, hi;
                        unpack2<KT>(w[e], lo, hi);
                        a = fmaf(lo, q[i][2 * e], a);
                        a = fmaf(hi, q[i][2 * e + 1], a);
                    }
                }
            }
            dot[u] = a;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int u = 0; u < kGroupsPerWarp; ++u) {
                dot[u] += __shfl_xor_sync(0xffffffffu, dot[u], o);
                kn_cur[u] += __shfl_xor_sync(0xffffffffu, kn_cur[u], o);
            }
        }
        if (lane < kGroupsPerWarp && t0 + lane < t_end) {
            float dsel = dot[0], ksel = kn_cur[0];
#pragma unroll
            for (int u = 1; u < kGroupsPerWarp; ++u) {
                if (lane == u) {
                    dsel = dot[u];
                    ksel = kn_cur[u];
                }
            }
            p.scores[(int64_t)li * p.n_groups + t0 + lane] = dsel / (qnorm * fmaxf(sqrtf(ksel), 1e-12f));
        }
        if (more) {
#pragma unroll
            for (int u = 0; u < kGroupsPerWarp; ++u) {
                kn_cur[u] = kn_nxt[u];
#pragma unroll
                for (int i = 0; i < NV; ++i) cur[u][i] = nxt[u][i];
            }
        }
    }
}

// Dot product of 8 adjacent channels of a stored k-bar (element `at` of the bank array) with 8 floats of q.
template <typename KT>
__device__ __forceinline__ float dot8(const void *rep_key, int64_t at, const float *q, float acc) {
    float k[8];
    load_meta8<KT>(rep_key, at, k);
    const float4 a = reinterpret_cast<const float4 *>(q)[0], b = reinterpret_cast<const float4 *>(q)[1];
    acc = fmaf(k[0], a.x, acc); acc = fmaf(k[1], a.y, acc); acc = fmaf(k[2], a.z, acc); acc = fmaf(k[3], a.w, acc);
    acc = fmaf(k[4], b.x, acc); acc = fmaf(k[5], b.y, acc); acc = fmaf(k[6], b.z, acc); acc = fmaf(k[7], b.w, acc);
    return acc;
}

// Scores of groups [t_begin, t_end) of layer li, by one block of kScoreWarps warps.  sq: the layer's question
// embedding (H*d floats) in shared memory, qn: its H squared norms.
// V4 > 0: PER_LAYER scoring with H*d == 128 * V4 and H <= 32 (the software-pipelined loop); V4 == 0: everything else.
template <int V4, typename KT>
__device__ __forceinline__ void score_block(const ScoreParams &p, const float *sq, const float *qn, int li, int t_begin,
                                            int t_end) {
    const int H = p.g.H, d = p.g.d, HD = H * d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if constexpr (V4 > 0) {
        score_groups_per_layer<V4, KT>(p, sq, qn, li, t_begin, t_end, warp, lane);
        return;
    }
    const int l = p.layer_begin + li;
    const float eps = 1e-12f;
#pragma unroll 1
    for (int t = t_begin + (V4 > 0 ? t_end : warp); t < t_end; t += kScoreWarps) {
        const int64_t slot = bank_slot(p.g, l, t, 0);
        if (!p.per_head) {
            float dot = 0.0f;
            for (int i = lane; i < HD / 8; i += 32) dot = dot8<KT>(p.rep_key, slot * d + i * 8, sq + i * 8, dot);
            float kn = 0.0f, qq = 0.0f;
            for (int hh = lane; hh < H; hh += 32) {
                kn += __ldg(p.rep_norm2 + slot + hh);
                qq += qn[hh];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                dot += __shfl_xor_sync(0xffffffffu, dot, o);
                kn += __shfl_xor_sync(0xffffffffu, kn, o);
                qq += __shfl_xor_sync(0xffffffffu, qq, o);
            }
            if (lane == 0)
                p.scores[(int64_t)li * p.n_groups + t] = dot / (fmaxf(sqrtf(qq), eps) * fmaxf(sqrtf(kn), eps));
        } else {
            for (int hh = 0; hh < H; ++hh) {
                float dot = 0.0f;
                for (int i = lane; i < d / 8; i += 32)
                    dot = dot8<KT>(p.rep_key, slot * d + hh * d + i * 8, sq + hh * d + i * 8, dot);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                if (lane == 0) {
                    const float kn = __ldg(p.rep_norm2 + slot + hh);
                    p.scores[((int64_t)li * H + hh) * p.n_groups + t] =
                        dot / (fmaxf(sqrtf(qn[hh]), eps) * fmaxf(sqrtf(kn), eps));
                }
            }
        }
    }
}


// grid (chunks, layer_count): block x scores groups [x * groups_per_block, (x+1) * groups_per_block) of its layer
template <int V4, typename KT>
__global__ void __launch_bounds__(kScoreWarps * 32) score_kernel(const ScoreParams p) {
    extern __shared__ __align__(16) float sq[];  // q of this layer: H*d floats, then H norms
    const int li = blockIdx.y, H = p.g.H, HD = H * p.g.d;
    grid_dependency_wait();  // the embeddings come from the kernel just ahead in the stream
    for (int i = threadIdx.x; i < HD; i += blockDim.x) sq[i] = p.qemb[(int64_t)li * HD + i];
    float *qn = sq + HD;
    if (threadIdx.x < H) qn[threadIdx.x] = p.qnorm2[(int64_t)li * H + threadIdx.x];
    __syncthreads();
    const int t_begin = blockIdx.x * p.groups_per_block;
    const int t_end = min(t_begin + p.groups_per_block, p.n_groups);
    score_block<V4, KT>(p, sq, qn, li, t_begin, t_end);
}

// The fast scoring loop exists for H*d = 128 * V4 with V4 in {1, 2, 4, 8}; a 16-bit k-bar needs H*d to be a multiple
// of 256.  Returns the V4 to instantiate, 0 for the general loop.
inline int score_fast_v4(int HD, bool fast, int meta_dtype) {
    if (!fast) return 0;
    if (HD != 128 && HD != 256 && HD != 512 && HD != 1024) return 0;
    if (meta_dtype != STOM_FP32 && HD == 128) return 0;
    return HD / 128;
}

}  // namespace stom
