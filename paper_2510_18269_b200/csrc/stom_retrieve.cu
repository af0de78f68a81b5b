// A2 + A3 in one launch, then A4: retrieval for one question (paper Sec. 3.4:
// similarity of the decoder state to every stored representative key, TopK,
// then reconstruction of the selected groups only; appendix "Question-guided
// single-pass retrieval" and "Cache reconstruction for decoding").
//
// The fused kernel runs with about two blocks per SM, each owning a
// contiguous run of one layer's stored groups:
//   prologue  the block builds the layer's question embedding q^(l) (mean
//             over the query heads of each GQA block and over the question
//             tokens) in shared memory -- Q of one layer is small and comes
//             from L2 for all but the first block that touches it; the rows
//             of several heads are in flight together, because this step is
//             memory latency -- and L2 bandwidth: every block of a layer wants
//             the same rows.  So the blocks of a layer are launched as
//             thread-block clusters: each block of a cluster embeds only its
//             share of the kv heads and the cluster exchanges the results
//             through distributed shared memory (one hardware cluster
//             barrier on each side of the exchange; no block returns before
//             them);
//   stream    cosine scores of the block's groups (the software-pipelined
//             loop of the stand-alone scoring kernel), written to `scores`;
//   select    every block takes a ticket on its layer's counter when its
//             scores are out; the block that draws the last ticket of a layer
//             selects that layer's top-K.  Nobody waits for anybody: a block
//             that is not last simply exits.  With enough workspace the
//             selection has two levels: each block first selects the top-K of
//             its own run (all blocks in parallel, a few keys per thread), and
//             the completing block only selects among chunks * K candidates,
//             which are in ascending index order, so ties still go to the
//             lower index and the result is the same set.
// The layer counters live in the caller's workspace and are zeroed by a
// memset enqueued ahead of the kernel; the selecting block also puts its
// counter back to zero.
#include "stom_async.cuh"
#include "stom_score.cuh"
#include "stom_topk.cuh"

namespace stom {

constexpr int kFusedThreads = kScoreWarps * 32;
constexpr int kFusedMaxKeys = 10240;  // rows up to this many scores are selected from shared memory

struct RetrieveParams {
    ScoreParams sp;
    int32_t k;
    int32_t *idx;          // [rows][k]
    uint32_t *counters;    // [layer_count], zero on entry
    int32_t keys_in_smem;  // the selecting block may stage a row's keys in shared memory
    // two-level selection (0: off): every block first selects the top-K of its own run of groups, the block
    // that completes the layer then selects among those candidates only
    int32_t two_level;
    int32_t *cand_idx;     // [layer_count][chunks][k] positions inside the block's run, ascending; unused -1
    float *cand_score;     // [layer_count][chunks][k] their scores; unused -inf
};

constexpr int kTwoLevelMaxK = 256;  // the selecting block keeps the chosen candidate positions in shared memory

constexpr int kEmbedHeadGroup = 4;  // kv heads whose rows are in flight together

// Raw 8 channels of one question row as loaded (16 bytes of a 16-bit type, 32 bytes of binary32).
template <typename T>
struct QRow {
    static constexpr int W = 8 * (int)sizeof(T) / 4;
    uint32_t w[W];
    __device__ __forceinline__ void load(const T *src) {
#pragma unroll
        for (int i = 0; i < W / 4; ++i) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src) + i);
            w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
        }
    }
    __device__ __forceinline__ void add_to(float (&acc)[8]) const {
        if constexpr (sizeof(T) == 4) {
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[c] += __uint_as_float(w[c]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float a, b;
                unpack2<T>(w[c], a, b);
                acc[2 * c] += a;
                acc[2 * c + 1] += b;
            }
        }
    }
};

// Question embedding of layer li for all kv heads, into sq[H*d] and qn[H] (shared memory).  A thread owns 8 adjacent
// channels; the rows of a head (rep * T_q of them) are dealt to RG = kFusedThreads / (d/8) row slots.  The heads go
// through in groups of kEmbedHeadGroup: a thread walks its rows of the whole group with kInFlight loads outstanding,
// whatever head they belong to, so the wait for memory is paid once or twice per group instead of once per head;
// part[head of the group][RG][d+4] combines the slots.  The call embeds heads h_first, h_first + h_step, ... only.
template <typename T>
__device__ __forceinline__ void embed_layer(const ScoreParams &p, int li, float *sq, float *qn, float *part,
                                            int h_first, int h_step) {
    constexpr int kInFlight = sizeof(T) == 4 ? 8 : 16;
    const int d = p.g.d, H = p.g.H, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lanes_per_row = d >> 3;
    const int RG = kFusedThreads / lanes_per_row;
    const int cq = tid % lanes_per_row, rs = tid / lanes_per_row;
    const int rows = p.rep * p.T_q, pitch = d + 4;
    const int per_head = (rows + RG - 1) / RG;  // rows of one head that a row slot walks
    const T *qbase = reinterpret_cast<const T *>(p.Q) + (int64_t)li * p.ql + cq * 8;
    const int n_mine = h_first < H ? (H - h_first + h_step - 1) / h_step : 0;  // heads this call embeds
    auto head_of = [&](int j) { return h_first + j * h_step; };                  // its j-th head
    for (int h0 = 0; h0 < n_mine; h0 += kEmbedHeadGroup) {
        const int hg = min(kEmbedHeadGroup, n_mine - h0);
        const int n_i = hg * per_head;
        float acc[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[c] = 0.0f;
        int cur = 0;  // head of the group that acc belongs to
        auto flush = [&](int hh) {
            float4 *mine = reinterpret_cast<float4 *>(part + (hh * RG + rs) * pitch + cq * 8);
            mine[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
            mine[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[c] = 0.0f;
        };
        // The walk i = 0 .. n_i-1 visits (head hh of the group, k-th row of this slot in that head); the row is
        // r = rs + k * RG = query head hr of the GQA block, token j.  All four are stepped, never divided out: an
        // integer division per load was a third of this prologue's instructions.
        const int hr0 = rs / p.T_q, j0 = rs - hr0 * p.T_q;
        int l_hh = 0, l_k = 0, l_hr = hr0, l_j = j0;  // state of the loading walk
        int a_hh = 0, a_k = 0;                        // state of the adding walk
        for (int i0 = 0; i0 < n_i; i0 += kInFlight) {
            QRow<T> x[kInFlight];
#pragma unroll
            for (int b = 0; b < kInFlight; ++b) {
#pragma unroll
                for (int j = 0; j < QRow<T>::W; ++j) x[b].w[j] = 0u;  // +0.0 in every format
                if (i0 + b < n_i) {
                    if (rs + l_k * RG < rows)
                        x[b].load(qbase + (int64_t)(head_of(h0 + l_hh) * p.rep + l_hr) * p.qh + (int64_t)l_j * p.qt);
                    if (++l_k == per_head) {  // next head of the group: back to the slot's first row
                        l_k = 0;
                        ++l_hh;
                        l_hr = hr0;
                        l_j = j0;
                    } else {
                        l_j += RG;
                        while (l_j >= p.T_q) {
                            l_j -= p.T_q;
                            ++l_hr;
                        }
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < kInFlight; ++b) {
                if (i0 + b < n_i) {
                    if (a_hh != cur) {
                        flush(cur);
                        cur = a_hh;
                    }
                    x[b].add_to(acc);
                    if (++a_k == per_head) {
                        a_k = 0;
                        ++a_hh;
                    }
                }
            }
        }
        flush(cur);
        __syncthreads();
        for (int e = tid; e < hg * d; e += kFusedThreads) {
            const int hh = e / d, c = e - hh * d;
            float a = 0.0f;
            for (int g = 0; g < RG; ++g) a += part[(hh * RG + g) * pitch + c];
            sq[head_of(h0 + hh) * d + c] = a / (float)rows;
        }
        __syncthreads();
        for (int hh = warp; hh < hg; hh += kFusedThreads / 32) {  // |q_h|^2: one warp per head
            float n2 = 0.0f;
            for (int c = lane; c < d; c += 32) {
                const float v = sq[head_of(h0 + hh) * d + c];
                n2 = fmaf(v, v, n2);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
            if (lane == 0) qn[head_of(h0 + hh)] = n2;
        }
        // part is rewritten by the next group only after that group's loads; the barrier below orders it for all
        __syncthreads();
    }
}

// grid (chunks, layer_count), kFusedThreads threads, optionally in clusters of consecutive chunks of a layer.
// Dynamic shared memory: q (H*d floats), norms (H rounded up to 4 floats), then a region used first as the embedding
// scratch and, in a selecting block, as the key array.
template <typename T, int V4, typename KT>
__global__ void __launch_bounds__(kFusedThreads) retrieve_kernel(const RetrieveParams rp) {
    extern __shared__ __align__(16) float dyn[];
    __shared__ TopkSmem tsm;
    __shared__ int s_last;
    const ScoreParams &p = rp.sp;
    const int li = blockIdx.y, H = p.g.H, HD = H * p.g.d, tid = threadIdx.x;
    float *sq = dyn, *qn = dyn + HD, *region = qn + ((H + 3) & ~3);

    grid_launch_dependents();  // the gather that follows may be scheduled as this grid drains; it waits before it reads idx
    // The blocks of a cluster (consecutive chunks of one layer) share the embedding: block r of C embeds heads
    // r, r + C, ... and fetches the others from their owners' shared memory.  Launched without clusters, C = 1.
    const uint32_t C = cluster_size(), r = cluster_rank();
    embed_layer<T>(p, li, sq, qn, region, (int)r, (int)C);
    if (C > 1) {
        cluster_sync();  // every block's heads are in its shared memory
        const int d4 = p.g.d >> 2;
        for (int e = tid; e < HD / 4; e += kFusedThreads) {
            const uint32_t owner = (uint32_t)(e / d4) % C;
            if (owner != r) reinterpret_cast<float4 *>(sq)[e] = ld_cluster_f4(reinterpret_cast<float4 *>(sq) + e, owner);
        }
        if (tid < H && (uint32_t)tid % C != r) qn[tid] = ld_cluster_f(qn + tid, (uint32_t)tid % C);
        cluster_sync();  // nobody leaves, or goes on to reuse its scratch, while a neighbour still reads from it
    }

    const int t_begin = blockIdx.x * p.groups_per_block;
    const int t_end = min(t_begin + p.groups_per_block, p.n_groups);
    score_block<V4, KT>(p, sq, qn, li, t_begin, t_end);

    uint32_t *skeys = reinterpret_cast<uint32_t *>(region);
    const int n = p.n_groups, chunks = gridDim.x;
    if (rp.two_level) {
        // ---- level 1: the candidates of this block's run
        __syncthreads();  // the run's scores are out (all warps of this block)
        const int64_t cbase = ((int64_t)li * chunks + blockIdx.x) * rp.k;
        const int len = t_end - t_begin;
        block_topk<kFusedThreads, kKeysRegs>(p.scores + (int64_t)li * n + t_begin, len, rp.k, rp.cand_idx + cbase,
                                             rp.cand_score + cbase, nullptr, skeys, tsm);
        for (int j = min(rp.k, len) + tid; j < rp.k; j += kFusedThreads) rp.cand_score[cbase + j] = -INFINITY;
    }

    // ---- ticket: the block that completes a layer selects its top-K
    __threadfence();  // this block's scores (and candidates) are visible device-wide before its ticket is
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&rp.counters[li], 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) rp.counters[li] = 0;  // as found
    if (rp.two_level) {
        // ---- level 2: among chunks * k candidates, kept in ascending index order
        __shared__ int32_t pos[kTwoLevelMaxK];
        const int ksel = min(rp.k, n);
        const int64_t cbase = (int64_t)li * chunks * rp.k;
        block_topk<kFusedThreads, kKeysRegs>(rp.cand_score + cbase, chunks * rp.k, ksel, pos, nullptr, nullptr, skeys, tsm);
        __syncthreads();
        int32_t *out = rp.idx + (int64_t)li * rp.k;
        for (int j = tid; j < rp.k; j += kFusedThreads) {
            int32_t g = -1;
            if (j < ksel) {
                const int c = pos[j] / rp.k;
                g = c * p.groups_per_block + __ldcg(rp.cand_idx + cbase + pos[j]);
            }
            out[j] = g;
        }
        return;
    }
    const int rows = p.per_head ? H : 1;
    for (int r = 0; r < rows; ++r) {
        const int64_t row = (int64_t)li * rows + r;
        const float *sc = p.scores + row * n;
        int32_t *out = rp.idx + row * rp.k;
        if (n <= kTopkRegKeys * kFusedThreads)
            block_topk<kFusedThreads, kKeysRegs>(sc, n, rp.k, out, nullptr, nullptr, skeys, tsm);
        else if (rp.keys_in_smem)
            block_topk<kFusedThreads, kKeysShared>(sc, n, rp.k, out, nullptr, nullptr, skeys, tsm);
        else
            block_topk<kFusedThreads, kKeysGlobal>(sc, n, rp.k, out, nullptr, nullptr, skeys, tsm);
        __syncthreads();  // the scratch is reused by the next row
    }
}

// Launch with thread-block clusters along x when `clusters` is set: the largest divisor of grid.x, up to the portable
// limit of 8, with which the whole grid is still resident at once (as it is without clusters); else single blocks.
template <typename KernelT>
static void launch_fused(KernelT kernel, const RetrieveParams &rp, dim3 grid, size_t smem, int clusters, cudaStream_t s) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = dim3(kFusedThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 1;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    for (int c = 8; clusters && c > 1; --c) {
        if (grid.x % c) continue;
        int resident = 0;
        at[0].val.clusterDim.x = (unsigned)c;
        if (cudaOccupancyMaxActiveClusters(&resident, kernel, &lc) == cudaSuccess &&
            (int64_t)resident * c >= (int64_t)grid.x * grid.y)
            break;
        (void)cudaGetLastError();
        at[0].val.clusterDim.x = 1;
    }
    (void)cudaLaunchKernelEx(&lc, kernel, rp);  // a failure is picked up by the caller's finish_launch()
}

template <typename T, typename KT>
static void launch_retrieve_kt(const RetrieveParams &rp, dim3 grid, size_t smem, int v4, int cluster, cudaStream_t s) {
    switch (v4) {
    case 4: launch_fused(retrieve_kernel<T, 4, KT>, rp, grid, smem, cluster, s); break;  // 4 kv heads x 128
    case 8: launch_fused(retrieve_kernel<T, 8, KT>, rp, grid, smem, cluster, s); break;  // 8 kv heads x 128
    case 2: launch_fused(retrieve_kernel<T, 2, KT>, rp, grid, smem, cluster, s); break;
    case 1:
        if constexpr (sizeof(KT) == 4) {
            launch_fused(retrieve_kernel<T, 1, KT>, rp, grid, smem, cluster, s);
            break;
        }
    default: launch_fused(retrieve_kernel<T, 0, KT>, rp, grid, smem, cluster, s); break;
    }
}

template <typename T>
static void launch_retrieve(const RetrieveParams &rp, dim3 grid, size_t smem, int HD, bool fast, int cluster,
                            cudaStream_t s) {
    const int md = rp.sp.g.meta_dtype, v4 = score_fast_v4(HD, fast, md);
    if (md == STOM_BF16) launch_retrieve_kt<T, __nv_bfloat16>(rp, grid, smem, v4, cluster, s);
    else if (md == STOM_FP16) launch_retrieve_kt<T, __half>(rp, grid, smem, v4, cluster, s);
    else launch_retrieve_kt<T, float>(rp, grid, smem, v4, cluster, s);
}

}  // namespace stom

using namespace stom;

// chunks the fused kernel cuts a layer into on a device with `sms` multiprocessors
static int retrieve_chunks(int sms, int layer_count, int n_groups) {
    int chunks = (2 * sms) / layer_count;
    if (chunks > (n_groups + 31) / 32) chunks = (n_groups + 31) / 32;
    return chunks < 1 ? 1 : chunks;
}

static int64_t up256(int64_t x) { return (x + 255) / 256 * 256; }

extern "C" int64_t stom_oqm_retrieve_workspace_bytes(const stom_oqm_config *cfg, int32_t layer_count,
                                                     int32_t n_groups, int32_t k) {
    if (check_config(cfg) || layer_count < 0 || n_groups < 0 || k < 1) return STOM_ERR_INVALID_ARG;
    const int64_t base = stom_oqm_score_workspace_bytes(cfg, layer_count);
    if (layer_count == 0 || k > kTwoLevelMaxK) return base;
    // sized for any device of up to 256 multiprocessors
    const int64_t chunks = retrieve_chunks(256, layer_count, n_groups);
    const int64_t two = up256((int64_t)layer_count * 4) + 2 * up256((int64_t)layer_count * chunks * k * 4);
    return two > base ? two : base;
}

extern "C" int32_t stom_oqm_retrieve(const stom_oqm_config *cfg, const stom_oqm_store *store,
                                     int32_t layer_begin, int32_t layer_count, int32_t n_groups,
                                     const void *Q, int32_t T_q, int64_t q_stride_layer,
                                     int64_t q_stride_head, int64_t q_stride_token,
                                     int32_t k, float *scores, int32_t *idx,
                                     void *k_active, void *v_active, int32_t out_dtype,
                                     int64_t stride_layer, int64_t stride_head, int64_t stride_token,
                                     int32_t token_offset, void *workspace, int64_t workspace_bytes,
                                     uint32_t *dev_flags, void *stream) {
    int32_t rc = check_config(cfg);
    if (rc) return rc;
    if ((rc = check_store(store))) return rc;
    if ((rc = check_layers(cfg, layer_begin, layer_count))) return rc;
    if (!Q || !scores || !idx || T_q < 1 || n_groups < 0 || k < 1) return STOM_ERR_INVALID_ARG;
    if (n_groups > cfg->capacity_groups) return STOM_ERR_CAPACITY;
    if (n_groups > (1 << 24)) return STOM_ERR_SHAPE;
    if (q_stride_layer < 0 || q_stride_head < 0 || q_stride_token < 0) return STOM_ERR_INVALID_ARG;
    if (!workspace || !aligned16(workspace) || workspace_bytes < stom_oqm_score_workspace_bytes(cfg, layer_count))
        return STOM_ERR_WORKSPACE;
    if (!aligned16(Q) || (reinterpret_cast<uintptr_t>(scores) & 3u) || (reinterpret_cast<uintptr_t>(idx) & 3u))
        return STOM_ERR_ALIGNMENT;
    const int dt = cfg->kv_dtype;
    if (!stride_ok(q_stride_layer, dt) || !stride_ok(q_stride_head, dt) || !stride_ok(q_stride_token, dt))
        return STOM_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (layer_count > 0 && n_groups > 0) {
        int dev = 0, sms = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaMemsetAsync(workspace, 0, (size_t)layer_count * sizeof(uint32_t), s);
        if (e != cudaSuccess) {
            set_last_cuda_error(e);
            return STOM_ERR_CUDA;
        }
        RetrieveParams rp;
        ScoreParams &p = rp.sp;
        p.Q = Q; p.ql = q_stride_layer; p.qh = q_stride_head; p.qt = q_stride_token;
        p.rep_key = store->rep_key; p.rep_norm2 = store->rep_norm2;
        p.qemb = nullptr; p.qnorm2 = nullptr;
        p.scores = scores;
        p.g = bank_geom(cfg);
        p.layer_begin = layer_begin; p.layer_count = layer_count; p.n_groups = n_groups; p.T_q = T_q;
        p.rep = cfg->n_q_heads / cfg->n_kv_heads;
        p.per_head = cfg->score_mode == STOM_SCORE_PER_HEAD;
        // one wave of about two blocks per SM; a block re-reads its layer's Q, so blocks are kept long
        int chunks = retrieve_chunks(sms, layer_count, n_groups);
        p.groups_per_block = (n_groups + chunks - 1) / chunks;
        chunks = (n_groups + p.groups_per_block - 1) / p.groups_per_block;
        rp.k = k; rp.idx = idx;
        rp.counters = static_cast<uint32_t *>(workspace);
        // two-level selection when it pays (several runs per layer, K well below a run) and the workspace has room
        const int64_t off_ci = up256((int64_t)layer_count * 4);
        const int64_t off_cs = off_ci + up256((int64_t)layer_count * chunks * k * 4);
        const int64_t need2 = off_cs + up256((int64_t)layer_count * chunks * k * 4);
        rp.two_level = !p.per_head && chunks >= 2 && k <= kTwoLevelMaxK && 2 * k <= p.groups_per_block &&
                       p.groups_per_block <= kTopkRegKeys * kFusedThreads &&
                       (int64_t)chunks * k <= kTopkRegKeys * kFusedThreads && workspace_bytes >= need2 &&
                       (reinterpret_cast<uintptr_t>(workspace) & 255u) == 0;
        rp.cand_idx = reinterpret_cast<int32_t *>(static_cast<uint8_t *>(workspace) + off_ci);
        rp.cand_score = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + off_cs);
        const int H = cfg->n_kv_heads, d = cfg->head_dim, HD = H * d;
        const int part_floats = (H < kEmbedHeadGroup ? H : kEmbedHeadGroup) * (kFusedThreads / (d / 8)) * (d + 4);
        const size_t fixed = (size_t)HD + ((H + 3) & ~3);
        int key_words = n_groups > kTopkRegKeys * kFusedThreads && n_groups <= kFusedMaxKeys ? n_groups : 0;
        if (sizeof(float) * (fixed + key_words) > 48 * 1024) key_words = 0;  // long rows are selected from global memory
        rp.keys_in_smem = key_words > 0;
        const size_t smem = sizeof(float) * (fixed + (part_floats > key_words ? part_floats : key_words));
        if (smem > 48 * 1024) return STOM_ERR_SHAPE;
        const dim3 grid((n_groups + p.groups_per_block - 1) / p.groups_per_block, layer_count);
        const bool fast = !p.per_head && H <= 32;
        const int cluster = grid.x > 1;  // several blocks per layer: let them share the embedding
        switch (dt) {
        case STOM_BF16: launch_retrieve<__nv_bfloat16>(rp, grid, smem, HD, fast, cluster, s); break;
        case STOM_FP16: launch_retrieve<__half>(rp, grid, smem, HD, fast, cluster, s); break;
        default: launch_retrieve<float>(rp, grid, smem, HD, fast, cluster, s); break;
        }
        if ((rc = finish_launch())) return rc;
    } else if (layer_count > 0) {
        // nothing stored: every slot of idx is unused
        const int32_t rows = layer_count * (cfg->score_mode == STOM_SCORE_PER_HEAD ? cfg->n_kv_heads : 1);
        rc = stom_oqm_topk(scores, rows, 0, 0, k, idx, nullptr, nullptr, stream);
        if (rc) return rc;
    }
    return dequant_gather_launch(cfg, store, layer_begin, layer_count, idx, k, n_groups, k_active, v_active, out_dtype,
                                 stride_layer, stride_head, stride_token, token_offset, dev_flags, stream,
                                 layer_count > 0 && n_groups > 0);
}
