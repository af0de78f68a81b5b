// Merge_{k_s} of Causal Temporal Reduction and the retained group (paper Sec. 3.3, the static half of the (G_d, G_s)
// equation, and the retained group G_t that holds both paths, |G_t| = G).  The paper consolidates the static tokens
// by a density-based clustering and fixes none of that method's parameters; the reading implemented here
// is the k-nearest-neighbour form of density-peak clustering (see include/stom_ctr.h for the rule, step by step).
//
// One block per frame.
//   Gram     all pairwise inner products of the frame's N feature rows: a [N x D] . [D x N] contraction, the one dense
//            product of CTR, on the tensor cores (mma.sync m16n8k16 on the 16-bit features, binary32 accumulation).
//            The rows arrive in shared memory in slabs of 64 channels (cp.async, a ring of four slabs, three on their
//            way while one is consumed; 16-byte columns swizzled by the row so that ldmatrix reads without bank
//            conflicts); only the 16 x 16 blocks on and below the diagonal are computed and a warp keeps the
//            accumulators of its blocks in registers over the whole contraction.  Squared distances d2(i,j) =
//            (|x_i|^2 + |x_j|^2 - 2 x_i.x_j) / D go to a packed triangle that takes the slabs' place.
//   cluster  a thread per token: density from the k nearest static neighbours, distance to the nearest denser token,
//            rank count of gamma = rho * delta for the centres, nearest centre for the rest -- a few passes over rows
//            of the triangle, N is a few hundred at most.
//   merge    a cluster's mean, 8 channels per thread, members in ascending token order, written straight into the
//            cluster's slot of the retained group; the selected dynamic rows are copied beside them.
#include "stom_internal.cuh"

#include "stom_ctr.h"

namespace stom {

constexpr int kMgThreads = 512;
constexpr int kMgWarps = kMgThreads / 32;
constexpr int kMgMaxTokens = 224;              // 14 row tiles of 16
constexpr int kMgMaxTiles = kMgMaxTokens / 16;
constexpr int kMgMaxBlocks = (kMgMaxTiles * (kMgMaxTiles + 1) / 2 + kMgWarps - 1) / kMgWarps;  // 16 x 16 blocks per warp
constexpr int kMgSlabCh = 64;                  // channels per slab: 128 bytes of a row
constexpr int kMgSlabs = 4;                    // slabs in the ring: three on their way while one is consumed
constexpr int kMgMaxKnn = 8;

struct MergeParams {
    const void *F;
    int64_t sf, st;  // element strides: frame, token
    const int32_t *k_s, *k_d, *static_idx, *dyn_idx;
    void *retained;
    int32_t *retained_pos, *centre, *assign;
    int32_t N, D, G, knn;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
template <typename T>
__device__ __forceinline__ void mg_mma(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1);
template <>
__device__ __forceinline__ void mg_mma<__nv_bfloat16>(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                      uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <>
__device__ __forceinline__ void mg_mma<__half>(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// position of d2(a, b) in the packed lower triangle
__device__ __forceinline__ int tri(int a, int b) { return a >= b ? a * (a + 1) / 2 + b : b * (b + 1) / 2 + a; }

// Shared-memory layout (bytes): the slab ring (later the triangle), then the per-token arrays
struct MergeLayout {
    int rows, slab_bytes, off_tri, off_nrm, off_rho, off_gam, off_slist, off_cid, off_clist, off_member, off_coff, off_slot,
        off_flag, total;
};
__host__ __device__ inline MergeLayout merge_layout(int N) {
    MergeLayout l;
    l.rows = (N + 15) / 16 * 16;
    l.slab_bytes = l.rows * kMgSlabCh * 2;
    // the triangle is written when the last slab has been consumed: it lies over the slabs
    const int slabs = kMgSlabs * l.slab_bytes, tri_bytes = l.rows * (l.rows + 1) / 2 * 4;
    l.off_tri = 0;
    int off = ((slabs > tri_bytes ? slabs : tri_bytes) + 127) / 128 * 128;
    l.off_nrm = off; off += l.rows * 4;
    l.off_rho = off; off += l.rows * 4;
    l.off_gam = off; off += l.rows * 4;
    l.off_slist = off; off += l.rows * 4;    // static tokens, ascending
    l.off_cid = off; off += l.rows * 4;      // per token: cluster id (static tokens), -1 otherwise
    l.off_clist = off; off += l.rows * 4;    // centre tokens, ascending
    l.off_member = off; off += l.rows * 4;   // static tokens ordered by cluster
    l.off_coff = off; off += (l.rows + 1) * 4;  // where each cluster's members start in `member`
    l.off_slot = off; off += l.rows * 4;     // retained slot of every cluster
    l.off_flag = off; off += l.rows;         // per token: 1 static, 3 centre
    l.total = (off + 15) / 16 * 16;
    return l;
}

template <typename T>
__global__ void __launch_bounds__(kMgThreads, 1) ctr_merge_kernel(const MergeParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int N = p.N, D = p.D, G = p.G, t = blockIdx.x;
    const MergeLayout L = merge_layout(N);
    const int NT = L.rows / 16;
    float *d2 = reinterpret_cast<float *>(smem + L.off_tri), *nrm = reinterpret_cast<float *>(smem + L.off_nrm);
    float *rho = reinterpret_cast<float *>(smem + L.off_rho), *gam = reinterpret_cast<float *>(smem + L.off_gam);
    int32_t *slist = reinterpret_cast<int32_t *>(smem + L.off_slist), *cid = reinterpret_cast<int32_t *>(smem + L.off_cid);
    int32_t *clist = reinterpret_cast<int32_t *>(smem + L.off_clist), *member = reinterpret_cast<int32_t *>(smem + L.off_member);
    int32_t *coff = reinterpret_cast<int32_t *>(smem + L.off_coff), *slot = reinterpret_cast<int32_t *>(smem + L.off_slot);
    unsigned char *flag = smem + L.off_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int k_s = p.k_s[t], k_d = p.k_d[t];
    const T *Ft = reinterpret_cast<const T *>(p.F) + (int64_t)t * p.sf;
    T *ret = reinterpret_cast<T *>(p.retained) + (int64_t)t * G * D;
    int32_t *rpos = p.retained_pos + (int64_t)t * G;

    // ---- the static list (ascending, -1 padded in global memory) and the per-token flags
    for (int i = tid; i < L.rows; i += kMgThreads) {
        flag[i] = 0;
        cid[i] = -1;
    }
    __syncthreads();
    int n_s = 0;
    for (int i = tid; i < N; i += kMgThreads) {
        const int s = p.static_idx[(int64_t)t * N + i];
        if (s >= 0 && s < N) {
            slist[i] = s;
            flag[s] = 1;
        }
    }
    for (int i = 0; i < N; i += 32) {  // every warp counts the list (it is dense from the front)
        const int s = i + lane < N ? p.static_idx[(int64_t)t * N + i + lane] : -1;
        n_s += __popc(__ballot_sync(0xffffffffu, s >= 0 && s < N));
    }
    __syncthreads();

    if (k_s > 0) {
        // ================================================================= Gram matrix on the tensor cores
        // 16 x 16 blocks (i, j), j <= i, numbered row by row; warp w owns a run of consecutive blocks, most of them in
        // one row, so that the row's operand fragment is loaded once per run of equal rows
        const int n_blk = NT * (NT + 1) / 2, per_warp = (n_blk + kMgWarps - 1) / kMgWarps;
        const int blk0 = warp * per_warp, n_mine_blk = max(0, min(per_warp, n_blk - blk0));
        int bi_[kMgMaxBlocks], bj_[kMgMaxBlocks];
        float acc[kMgMaxBlocks][2][4];
#pragma unroll
        for (int b = 0; b < kMgMaxBlocks; ++b) {
            const int n = blk0 + b;
            int i = 0;
            while ((i + 1) * (i + 2) / 2 <= n) ++i;  // row of block n
            bi_[b] = i;
            bj_[b] = n - i * (i + 1) / 2;
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[b][u][e] = 0.0f;
        }
        const uint32_t slab0 = (uint32_t)__cvta_generic_to_shared(smem);
        // rows beyond N stay zero in every slab
        for (int e = tid; e < (L.rows - N) * 8 * kMgSlabs; e += kMgThreads) {
            const int sl = e / ((L.rows - N) * 8), r = N + (e % ((L.rows - N) * 8)) / 8, c = e % 8;
            *reinterpret_cast<uint4 *>(smem + sl * L.slab_bytes + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
        }
        // Where a lane's ldmatrix row sits inside a tile, per k-step of a slab: the left operand's lane l supplies row
        // l % 16 and the 16-byte column 2 ks + l / 16; the right operand's, row l % 8 + 8 (l / 16) and column 2 ks +
        // (l / 8) % 2.  A tile starts at a multiple of 16 rows, so the swizzle (column ^ row % 8) depends on the lane only.
        uint32_t offA[kMgSlabCh / 16], offB[kMgSlabCh / 16];
#pragma unroll
        for (int ks = 0; ks < kMgSlabCh / 16; ++ks) {
            const int ra = lane & 15, ca = 2 * ks + (lane >> 4);
            const int rb = (lane & 7) + ((lane >> 4) << 3), cb = 2 * ks + ((lane >> 3) & 1);
            offA[ks] = (uint32_t)(ra * 128 + ((ca ^ (ra & 7)) << 4));
            offB[ks] = (uint32_t)(rb * 128 + ((cb ^ (rb & 7)) << 4));
        }
        const int n_chunks = D / kMgSlabCh;
        // channels [64 chunk, 64 chunk + 64) of rows 0 .. N-1 into slab chunk % kMgSlabs; always one group per call, an
        // empty one past the last chunk, so that the number of groups in flight tells which chunk has landed
        auto load_slab = [&](int chunk) {
            if (chunk < n_chunks) {
                const uint32_t to = slab0 + (chunk % kMgSlabs) * L.slab_bytes;
                for (int e = tid; e < N * 8; e += kMgThreads) {
                    const int r = e >> 3, c = e & 7;
                    cp_async16(to + r * 128 + ((c ^ (r & 7)) << 4), Ft + (int64_t)r * p.st + chunk * kMgSlabCh + c * 8);
                }
            }
            cp_async_commit();
        };
        for (int ch = 0; ch < kMgSlabs - 1; ++ch) load_slab(ch);
        for (int ch = 0; ch < n_chunks; ++ch) {
            cp_async_wait<kMgSlabs - 2>();  // chunk ch has landed (this thread's part of it)
            __syncthreads();                // ... everybody's; and everybody is done with chunk ch - 1
            load_slab(ch + kMgSlabs - 1);   // into the slab chunk ch - 1 has just left
            const uint32_t base = slab0 + (ch % kMgSlabs) * L.slab_bytes;
#pragma unroll
            for (int ks = 0; ks < kMgSlabCh / 16; ++ks) {
                const uint32_t pa = base + offA[ks], pb = base + offB[ks];
                uint32_t a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
                for (int b = 0; b < kMgMaxBlocks; ++b) {
                    if (b < n_mine_blk) {  // warp-uniform
                        uint32_t b0, b1, b2, b3;
                        if (b == 0 || bi_[b] != bi_[b - 1])  // (warp-uniform) a tile of 16 rows is 2048 bytes of a slab
                            ldmatrix_x4(pa + (bi_[b] << 11), a0, a1, a2, a3);
                        ldmatrix_x4(pb + (bj_[b] << 11), b0, b1, b2, b3);
                        mg_mma<T>(acc[b][0], a0, a1, a2, a3, b0, b1);
                        mg_mma<T>(acc[b][1], a0, a1, a2, a3, b2, b3);
                    }
                }
            }
        }
        cp_async_wait<0>();
        __syncthreads();  // the slabs are dead: the triangle takes their place
        // ---- squared norms from the diagonal blocks, then the distances
        const int g = lane >> 2, tq = lane & 3;
#pragma unroll
        for (int b = 0; b < kMgMaxBlocks; ++b) {
            if (b < n_mine_blk && bi_[b] == bj_[b]) {
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int r = g + 8 * (e >> 1), c = 8 * u + 2 * tq + (e & 1);
                        if (r == c) nrm[16 * bi_[b] + r] = acc[b][u][e];
                    }
            }
        }
        __syncthreads();
        const float inv_d = 1.0f / (float)D;
#pragma unroll
        for (int b = 0; b < kMgMaxBlocks; ++b) {
            if (b < n_mine_blk) {
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int r = 16 * bi_[b] + g + 8 * (e >> 1), c = 16 * bj_[b] + 8 * u + 2 * tq + (e & 1);
                        if (c <= r) d2[r * (r + 1) / 2 + c] = fmaxf(0.0f, (nrm[r] + nrm[c]) - 2.0f * acc[b][u][e]) * inv_d;
                    }
            }
        }
        __syncthreads();

        // ================================================================= density peaks: two threads per static token
        // (n_s <= N <= kMgMaxTokens, 2 * kMgMaxTokens <= kMgThreads: thread 2a + h takes the candidates b = h, h + 2, ...
        // of token a; the two are neighbours in a warp and combine by shuffle)
        static_assert(2 * kMgMaxTokens <= kMgThreads, "two threads per token");
        const int kk = min(p.knn, n_s - 1);
        const int a = tid >> 1, hf = tid & 1;
        const bool mine = a < n_s;
        const int ia = mine ? slist[a] : 0, row = ia * (ia + 1) / 2;
        float far2 = 0.0f;  // the token's largest squared distance to another static token
        {
            float best[kMgMaxKnn];  // the smallest squared distances among this thread's candidates, ascending
#pragma unroll
            for (int q = 0; q < kMgMaxKnn; ++q) best[q] = INFINITY;
            if (mine) {
#pragma unroll 4
                for (int b = hf; b < n_s; b += 2) {
                    const int ib = slist[b];
                    float v = d2[ib <= ia ? row + ib : ib * (ib + 1) / 2 + ia];
                    far2 = fmaxf(far2, v);          // (the token itself adds 0)
                    v = b == a ? INFINITY : v;      // ... and is no neighbour of itself
#pragma unroll
                    for (int q = 0; q < kMgMaxKnn; ++q) {  // insertion: v sinks to its place, the largest falls out
                        const float lo = fminf(best[q], v);
                        v = fmaxf(best[q], v);
                        best[q] = lo;
                    }
                }
            }
            // the partner's list sinks into this one: both threads end with the smallest of all candidates
            float theirs[kMgMaxKnn];
#pragma unroll
            for (int q = 0; q < kMgMaxKnn; ++q) theirs[q] = __shfl_xor_sync(0xffffffffu, best[q], 1);
            far2 = fmaxf(far2, __shfl_xor_sync(0xffffffffu, far2, 1));
#pragma unroll
            for (int e = 0; e < kMgMaxKnn; ++e) {
                float v = theirs[e];
#pragma unroll
                for (int q = 0; q < kMgMaxKnn; ++q) {
                    const float lo = fminf(best[q], v);
                    v = fmaxf(best[q], v);
                    best[q] = lo;
                }
            }
            float sum = 0.0f;
#pragma unroll
            for (int q = 0; q < kMgMaxKnn; ++q)
                if (q < kk) sum += best[q];
            if (mine && hf == 0) rho[a] = kk > 0 ? expf(-sum / (float)kk) : 1.0f;
        }
        __syncthreads();
        {
            const float ra = mine ? rho[a] : 0.0f;
            float near2 = INFINITY;
            if (mine) {
#pragma unroll 4
                for (int b = hf; b < n_s; b += 2) {  // (b == a is never denser than a)
                    const int ib = slist[b];
                    const float rb = rho[b], v = d2[ib <= ia ? row + ib : ib * (ib + 1) / 2 + ia];
                    near2 = (rb > ra || (rb == ra && b < a)) ? fminf(near2, v) : near2;
                }
            }
            near2 = fminf(near2, __shfl_xor_sync(0xffffffffu, near2, 1));
            if (mine && hf == 0) gam[a] = ra * sqrtf(near2 == INFINITY ? far2 : near2);
        }
        __syncthreads();
        // the k_s tokens of largest gamma (rank count; the earlier token among equals), in ascending token order
        {
            const float ga = mine ? gam[a] : 0.0f;
            int rank = 0;
            if (mine)
                for (int b = hf; b < n_s; b += 2) rank += gam[b] > ga || (gam[b] == ga && b < a);
            rank += __shfl_xor_sync(0xffffffffu, rank, 1);
            if (mine && hf == 0 && rank < k_s) flag[ia] = 3;
        }
        __syncthreads();
        for (int a = tid; a < n_s; a += kMgThreads) {
            if (flag[slist[a]] == 3) {
                int before = 0;
                for (int b = 0; b < a; ++b) before += flag[slist[b]] == 3;
                clist[before] = slist[a];
                cid[slist[a]] = before;
            }
        }
        __syncthreads();
        // every other static token joins its nearest centre (the earlier centre among equals)
        for (int a = tid; a < n_s; a += kMgThreads) {
            const int ia = slist[a];
            if (flag[ia] != 3) {
                int best = 0;
                float bd = d2[tri(ia, clist[0])];
                for (int j = 1; j < k_s; ++j) {
                    const float v = d2[tri(ia, clist[j])];
                    if (v < bd) {
                        bd = v;
                        best = j;
                    }
                }
                cid[ia] = best;
            }
        }
        __syncthreads();
        // members ordered by cluster, ascending token inside a cluster (counting passes)
        for (int j = tid; j <= k_s; j += kMgThreads) {
            int n = 0;
            for (int a = 0; a < n_s; ++a) n += cid[slist[a]] < j;
            coff[j] = n;
        }
        __syncthreads();
        for (int a = tid; a < n_s; a += kMgThreads) {
            const int c = cid[slist[a]];
            int within = 0;
            for (int b = 0; b < a; ++b) within += cid[slist[b]] == c;
            member[coff[c] + within] = slist[a];
        }
    }
    __syncthreads();

    // ================================================================= the retained group, in position order
    // slot of dynamic token number a = a + centres before it; slot of centre j = j + dynamic tokens before it
    const int32_t *dyn = p.dyn_idx + (int64_t)t * G;
    int32_t *dslot = reinterpret_cast<int32_t *>(gam);  // (gamma is not needed any more)
    for (int a = tid; a < k_d; a += kMgThreads) {
        const int tok = dyn[a];
        int before = 0;
        for (int j = 0; j < k_s; ++j) before += clist[j] < tok;
        rpos[a + before] = tok;
        dslot[a] = a + before;
    }
    for (int j = tid; j < k_s; j += kMgThreads) {
        int before = 0;
        for (int a = 0; a < k_d; ++a) before += dyn[a] < clist[j];
        slot[j] = j + before;
        rpos[j + before] = clist[j];
    }
    for (int w = k_d + k_s + tid; w < G; w += kMgThreads) rpos[w] = -1;
    if (p.centre)
        for (int j = tid; j < G; j += kMgThreads) p.centre[(int64_t)t * G + j] = j < k_s ? clist[j] : -1;
    if (p.assign)
        for (int a = tid; a < N; a += kMgThreads) p.assign[(int64_t)t * N + a] = a < n_s && k_s > 0 ? cid[slist[a]] : -1;
    __syncthreads();
    const int vec = D / 8;  // 16-byte vectors of a row
    for (int e = tid; e < k_d * vec; e += kMgThreads) {
        const int a = e / vec, c = e - a * vec;
        reinterpret_cast<uint4 *>(ret + (int64_t)dslot[a] * D)[c] = __ldg(reinterpret_cast<const uint4 *>(Ft + (int64_t)dyn[a] * p.st) + c);
    }
    for (int e = tid; e < (G - k_d - k_s) * vec; e += kMgThreads) {
        const int w = k_d + k_s + e / vec, c = e % vec;
        reinterpret_cast<uint4 *>(ret + (int64_t)w * D)[c] = make_uint4(0, 0, 0, 0);
    }
    // a cluster's mean: 8 channels per thread, the members added up in ascending token order
    for (int e = tid; e < k_s * vec; e += kMgThreads) {
        const int j = e / vec, c = e - j * vec;
        float s8[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) s8[q] = 0.0f;
        const int m0 = coff[j], m1 = coff[j + 1];
        for (int m = m0; m < m1; m += 4) {  // the loads of four members are in flight together; added in member order
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = m + u < m1 ? __ldg(reinterpret_cast<const uint4 *>(Ft + (int64_t)member[m + u] * p.st) + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (m + u < m1) {
                    const uint32_t w4[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float lo, hi;
                        unpack2<T>(w4[q], lo, hi);
                        s8[2 * q] += lo;
                        s8[2 * q + 1] += hi;
                    }
                }
            }
        }
        // true division: the binary32 sum of a few 16-bit values is exact, so the quotient is the correctly rounded mean
        const float cnt = (float)(m1 - m0);
        uint4 o;
        o.x = pack2<T>(__fdiv_rn(s8[0], cnt), __fdiv_rn(s8[1], cnt));
        o.y = pack2<T>(__fdiv_rn(s8[2], cnt), __fdiv_rn(s8[3], cnt));
        o.z = pack2<T>(__fdiv_rn(s8[4], cnt), __fdiv_rn(s8[5], cnt));
        o.w = pack2<T>(__fdiv_rn(s8[6], cnt), __fdiv_rn(s8[7], cnt));
        reinterpret_cast<uint4 *>(ret + (int64_t)slot[j] * D)[c] = o;
    }
}

}  // namespace stom

using namespace stom;

extern "C" int32_t stom_ctr_merge(const void *F, int32_t dtype, int32_t T, int32_t N, int32_t D, int64_t stride_frame,
                                  int64_t stride_token, const int32_t *k_s, const int32_t *k_d, const int32_t *static_idx,
                                  const int32_t *dyn_idx, int32_t G, int32_t knn, void *retained, int32_t *retained_pos,
                                  int32_t *centre, int32_t *assign, void *stream) {
    if (!F || !k_s || !k_d || !static_idx || !dyn_idx || !retained || !retained_pos || T < 0 || N < 1 || D < 1 || G < 1 || knn < 0)
        return STOM_ERR_INVALID_ARG;
    if (dtype != STOM_BF16 && dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    if (G > N || N > kMgMaxTokens || D % kMgSlabCh || D > 8192 || knn > kMgMaxKnn) return STOM_ERR_SHAPE;
    if (stride_token < D || stride_frame < 0) return STOM_ERR_INVALID_ARG;
    if (!aligned16(F) || !aligned16(retained) || !stride_ok(stride_frame, dtype) || !stride_ok(stride_token, dtype))
        return STOM_ERR_ALIGNMENT;
    const void *ptrs[7] = {k_s, k_d, static_idx, dyn_idx, retained_pos, centre, assign};
    for (const void *q : ptrs)
        if (reinterpret_cast<uintptr_t>(q) & 3u) return STOM_ERR_ALIGNMENT;
    if (T == 0) return STOM_OK;
    MergeParams p{F, stride_frame, stride_token, k_s, k_d, static_idx, dyn_idx, retained, retained_pos, centre, assign, N, D, G, knn};
    const size_t smem = (size_t)merge_layout(N).total;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (dtype == STOM_BF16) {
        e = cudaFuncSetAttribute(ctr_merge_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) ctr_merge_kernel<__nv_bfloat16><<<(unsigned)T, kMgThreads, smem, s>>>(p);
    } else {
        e = cudaFuncSetAttribute(ctr_merge_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) ctr_merge_kernel<__half><<<(unsigned)T, kMgThreads, smem, s>>>(p);
    }
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    return finish_launch();
}

extern "C" int32_t stom_ctr_reduce_tokens(const void *F, const void *prev, int32_t dtype, int32_t T, int32_t N, int32_t D,
                                          int64_t stride_frame, int64_t stride_token, const float *alpha, int32_t G,
                                          float tau_c, int32_t knn, float *sim, int32_t *k_s, int32_t *k_d,
                                          int32_t *static_idx, int32_t *dyn_idx, void *retained, int32_t *retained_pos,
                                          void *stream) {
    // every argument list is checked before the first launch
    if (!retained || !retained_pos || knn < 0) return STOM_ERR_INVALID_ARG;
    if (dtype != STOM_BF16 && dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    if (N < 1 || G < 1 || G > N || N > kMgMaxTokens || D < 1 || D % kMgSlabCh || D > 8192 || knn > kMgMaxKnn) return STOM_ERR_SHAPE;
    if (!aligned16(retained) || (reinterpret_cast<uintptr_t>(retained_pos) & 3u)) return STOM_ERR_ALIGNMENT;
    int32_t rc = stom_ctr_reduce(F, prev, dtype, T, N, D, stride_frame, stride_token, alpha, G, tau_c, sim, k_s, k_d,
                                 static_idx, dyn_idx, stream);
    if (rc) return rc;
    return stom_ctr_merge(F, dtype, T, N, D, stride_frame, stride_token, k_s, k_d, static_idx, dyn_idx, G, knn, retained,
                          retained_pos, nullptr, nullptr, stream);
}
