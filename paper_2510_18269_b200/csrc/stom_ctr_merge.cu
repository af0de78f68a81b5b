// Merge_{k_s} of Causal Temporal Reduction and the retained group (paper Sec. 3.3, the static half of the (G_d, G_s)
// equation, and the retained group G_t that holds both paths, |G_t| = G).  The paper consolidates the static tokens
// by a density-based clustering and fixes none of that method's parameters; the reading implemented here
// is the k-nearest-neighbour form of density-peak clustering (see include/stom_ctr.h for the rule, step by step).
//
// One block of 16 warps per frame, two blocks per multiprocessor: the tensor memory a block's Gram stage needs is
// allocated when that stage starts and given back as soon as the accumulators are read, so the blocks of a
// multiprocessor take turns at it and one frame's load-bound Gram stage runs beside another's clustering.
//   Gram     all pairwise inner products of the frame's N feature rows: a [N x D] . [D x N] contraction, the one dense
//            product of CTR, on the fifth-generation tensor cores (tcgen05.mma, kind::f16, binary32 accumulators in
//            tensor memory).  The rows arrive in shared memory in slabs of 64 channels (cp.async, a ring of slabs) in
//            the canonical K-major layout with 128-byte swizzle -- a row is 128 bytes, its 16-byte columns XOR-ed
//            with the row number modulo 8 -- so the same slab is both operands: the left one is a tile of 128 rows
//            (rows 0..127, and a second tile that ends at the last row), the right one all rows.  One thread issues
//            the products of a slab (4 steps of 16 channels x 2 tiles) and commits them to the slab's mbarrier, on
//            which the loaders wait before they refill the slab.  When the last slab's products have completed, the
//            16 warps read the accumulators from tensor memory (a warp reaches the 32 lanes of its quarter), and the
//            squared distances d2(i,j) = (|x_i|^2 + |x_j|^2 - 2 x_i.x_j) / D, j <= i, go to a packed triangle that
//            takes the slabs' place.
//   cluster  two threads per static token (neighbours in a warp, combined by shuffle): density from the k nearest
//            static neighbours, distance to the nearest denser token, rank count of gamma = rho * delta for the
//            centres, nearest centre for the rest -- a few passes over rows of the triangle.  Orders and places
//            (the centres in token order, a member's place in its cluster) come from warp ballots and matches over 32
//            consecutive tokens and a small table of per-warp counts, never from a thread walking all tokens.
//   merge    a cluster's mean, 8 channels per thread, members in ascending token order, written straight into the
//            cluster's slot of the retained group; the selected dynamic rows are copied beside them.
#include <type_traits>

#include "stom_async.cuh"
#include "stom_internal.cuh"

#include "stom_ctr.h"

namespace stom {

constexpr int kMgThreads = 512;
constexpr int kMgWarps = kMgThreads / 32;
constexpr int kMgMaxTokens = 224;              // 14 row tiles of 16
constexpr int kMgTmemCols = 512;               // tile 0: 128 columns, tile 1: up to 224; a power of two
constexpr unsigned long long kMgWaitLimitNs = 100000000ull;  // a product that has not completed after 0.1 s ends the block
constexpr int kMgSlabCh = 64;                  // channels per slab: 128 bytes of a row
constexpr int kMgSlabs = 3;                    // slabs in the ring: two on their way while one is consumed
constexpr int kMgMaxKnn = 8;

struct MergeParams {
    const void *F;
    int64_t sf, st;  // element strides: frame, token
    const int32_t *k_s, *k_d, *static_idx, *dyn_idx;
    void *retained;
    int32_t *retained_pos, *centre, *assign;
    int32_t N, D, G, knn;
    uint32_t *flags;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// ---- tcgen05: tensor memory and the matrix product that reads both operands from shared memory
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {  // one whole warp; writes the base address
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {  // the same warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// writes of the generic proxy (cp.async, plain stores) become visible to the asynchronous proxy (the tensor cores)
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Shared-memory matrix descriptor of a K-major operand in the 128-byte-swizzle layout: rows of 128 bytes, groups of 8
// rows 1024 bytes apart; `addr` is where the tile starts (a multiple of 1024) plus 32 bytes per step of 16 channels.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t addr) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: binary32 accumulator, both operands of type `fmt` (0 fp16, 1 bf16) and K-major,
// a tile of 128 rows by n columns
__device__ __forceinline__ uint32_t umma_idesc(uint32_t fmt, uint32_t n) {
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
// D[tmem] (+)= A[smem] . B[smem]^T, issued by one thread
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// all products issued so far by this thread arrive (once) on the mbarrier when they have completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive accumulator columns of this thread's lane (row) of tensor memory
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, "
        "%18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// position of d2(a, b) in the packed lower triangle
__device__ __forceinline__ int tri(int a, int b) { return a >= b ? a * (a + 1) / 2 + b : b * (b + 1) / 2 + a; }

// Shared-memory layout (bytes): the slab ring (later the triangle), then the per-token arrays
struct MergeLayout {
    int rows, slab_bytes, off_tri, off_nrm, off_rho, off_gam, off_slist, off_cid, off_clist, off_member, off_coff, off_slot,
        off_flag, off_wcnt, off_bar, total;
};
__host__ __device__ inline MergeLayout merge_layout(int N) {
    MergeLayout l;
    l.rows = (N + 15) / 16 * 16;
    // a slab holds at least the 128 rows a tile of the left operand spans (rows past the frame's are never used)
    l.slab_bytes = (l.rows > 128 ? l.rows : 128) * kMgSlabCh * 2;
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
    off = (off + 15) / 16 * 16;
    l.off_wcnt = off; off += (kMgMaxTokens / 32) * l.rows * 4;  // [warp of 32 static tokens][cluster]: members it holds
    l.off_bar = off; off += kMgSlabs * 8 + 16;  // one mbarrier per slab, the tensor-memory base address, the abort word
    l.total = (off + 15) / 16 * 16;
    return l;
}

template <typename T>
__global__ void __launch_bounds__(kMgThreads, 2) ctr_merge_kernel(const MergeParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
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
        // Tile 0 of the left operand is rows 0..127, tile 1 the 128 rows that end at the last one (they overlap where
        // the frame has fewer than 256 rows; a frame of up to 128 rows has tile 0 only).  The right operand is all rows.
        const uint32_t slab0 = smem_u32(smem), bar0 = smem_u32(smem + L.off_bar);
        volatile uint32_t *tmem_word = reinterpret_cast<volatile uint32_t *>(smem + L.off_bar + kMgSlabs * 8);
        volatile uint32_t *abort_flag = tmem_word + 1;
        const bool two_tiles = L.rows > 128;
        const int R1 = L.rows - 128;  // first row of tile 1 (a multiple of 16)
        const bool aligned = (slab0 & 1023u) == 0;  // the swizzle is a function of the address: slabs start on 1024 bytes
        if (tid == 0) {
            for (int sl = 0; sl < kMgSlabs; ++sl) mbar_init(bar0 + 8 * sl, 1);
            // (a frame is not started on the tensor cores once another frame of the call has given up)
            const bool gave_up = p.flags && (*reinterpret_cast<volatile uint32_t *>(p.flags) & STOM_FLAG_TIMEOUT);
            *abort_flag = aligned && !gave_up ? 0u : 1u;
            mbar_init_fence();
        }
        if (warp == 0) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_word)), kMgTmemCols);
        // rows beyond N stay zero in every slab (their products are never read, but they must be numbers)
        for (int e = tid; e < (L.slab_bytes / 128 - N) * 8 * kMgSlabs; e += kMgThreads) {
            const int per = (L.slab_bytes / 128 - N) * 8;
            const int sl = e / per, r = N + (e % per) / 8, c = e % 8;
            *reinterpret_cast<uint4 *>(smem + sl * L.slab_bytes + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        const uint32_t tmem = *tmem_word;
        bool dead = *abort_flag != 0;
        if (dead && tid == 0 && p.flags) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
        const int n_chunks = D / kMgSlabCh;
        // channels [64 chunk, 64 chunk + 64) of rows 0 .. N-1 into slab chunk % kMgSlabs; always one group per call, an
        // empty one past the last chunk, so that the number of groups in flight tells which chunk has landed
        auto load_slab = [&](int chunk) {
            if (chunk < n_chunks && !dead) {
                const uint32_t to = slab0 + (chunk % kMgSlabs) * L.slab_bytes;
                for (int e = tid; e < N * 8; e += kMgThreads) {
                    const int r = e >> 3, c = e & 7;
                    cp_async16(to + r * 128 + ((c ^ (r & 7)) << 4), Ft + (int64_t)r * p.st + chunk * kMgSlabCh + c * 8);
                }
            }
            cp_async_commit();
        };
        const uint32_t fmt = sizeof(T) == 2 && std::is_same<T, __nv_bfloat16>::value ? 1u : 0u;
        const uint32_t idesc0 = umma_idesc(fmt, 128u < (uint32_t)L.rows ? 128u : (uint32_t)L.rows);
        const uint32_t idesc1 = umma_idesc(fmt, (uint32_t)L.rows);
        for (int ch = 0; ch < kMgSlabs - 1; ++ch) load_slab(ch);
        for (int ch = 0; ch < n_chunks; ++ch) {
            cp_async_wait<kMgSlabs - 2>();  // chunk ch has landed (this thread's part of it)
            fence_proxy_async();            // ... and the tensor cores may read it
            __syncthreads();                // ... everybody's
            if (tid == 0 && !dead) {
                tc_fence_after_sync();
                const uint32_t base = slab0 + (ch % kMgSlabs) * L.slab_bytes;
#pragma unroll
                for (int ks = 0; ks < kMgSlabCh / 16; ++ks) {
                    const uint64_t b = umma_desc_k128(base + ks * 32);
                    const uint32_t acc = (ch | ks) != 0;
                    umma_ss(tmem, b, b, idesc0, acc);  // rows 0..127 against columns 0..127 (only j <= i is read)
                    if (two_tiles) umma_ss(tmem + 128, umma_desc_k128(base + R1 * 128 + ks * 32), b, idesc1, acc);
                }
                umma_commit(bar0 + 8 * (ch % kMgSlabs));  // arrives when these products no longer need the slab
            }
            // the slab of chunk ch - 1 takes chunk ch + kMgSlabs - 1 once that chunk's products have completed
            if (ch > 0 && ch + kMgSlabs - 1 < n_chunks && !dead) {
                const int pc = ch - 1;
                if (!mbar_wait_bounded(bar0 + 8 * (pc % kMgSlabs), (pc / kMgSlabs) & 1, abort_flag, kMgWaitLimitNs)) {
                    dead = true;
                    *abort_flag = 1;  // everybody else's waits end at once
                }
            }
            load_slab(ch + kMgSlabs - 1);
        }
        cp_async_wait<0>();
        // every product has completed when the last chunk's have (a commit covers all products issued before it)
        if (!dead) {
            const int lc = n_chunks - 1;
            if (!mbar_wait_bounded(bar0 + 8 * (lc % kMgSlabs), (lc / kMgSlabs) & 1, abort_flag, kMgWaitLimitNs)) {
                dead = true;
                *abort_flag = 1;
            }
        }
        if (dead) {
            *abort_flag = 1;
            if (p.flags && (tid & 31) == 0) atomicOr(p.flags, STOM_FLAG_TIMEOUT);
        }
        tc_fence_after_sync();
        __syncthreads();  // the slabs are dead: the triangle takes their place
        dead = *abort_flag != 0;

        // ---- a warp reaches lanes 32 q .. 32 q + 31 of tensor memory, q = warp % 4: lane l of the warp is row 32 q + l of
        //      tile 0 and row R1 + 32 q + l of tile 1; the four warps of a quarter share out the blocks of 32 columns
        const int q = warp & 3, jw = warp >> 2;
        const uint32_t lane_base = tmem + ((uint32_t)(32 * q) << 16);
        const int r0 = 32 * q + lane, r1 = R1 + 32 * q + lane;  // this thread's row in tile 0 and in tile 1
        float v[32];
        if (!dead) {
            // squared norms from the diagonal: row r of tile 0 for r < 128, of tile 1 above
            if (jw == 0 && 32 * q < L.rows) {
                tmem_ld32(lane_base + 32 * q, v);
                float dg = 0.0f;
#pragma unroll
                for (int i = 0; i < 32; ++i) dg = i == lane ? v[i] : dg;
                if (r0 < N) nrm[r0] = dg;
            }
            if (jw == 1 && two_tiles) {
                tmem_ld32(lane_base + 128 + R1 + 32 * q, v);
                float dg = 0.0f;
#pragma unroll
                for (int i = 0; i < 32; ++i) dg = i == lane ? v[i] : dg;
                if (r1 >= 128 && r1 < N) nrm[r1] = dg;
            }
        }
        __syncthreads();
        if (!dead) {
            const float inv_d = 1.0f / (float)D;
            // tile 0: rows 32 q .. 32 q + 31 need column blocks 0 .. q
            for (int cb = jw; cb <= q && 32 * q < L.rows; cb += 4) {
                tmem_ld32(lane_base + 32 * cb, v);
                if (r0 < N) {
                    const float nr = nrm[r0];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int c = 32 * cb + i;
                        if (c <= r0) d2[r0 * (r0 + 1) / 2 + c] = fmaxf(0.0f, (nr + nrm[c]) - 2.0f * v[i]) * inv_d;
                    }
                }
            }
            // tile 1: rows R1 + 32 q .. need column blocks 0 .. (R1 + 32 q + 31) / 32; only rows from 128 on are new
            if (two_tiles && R1 + 32 * q + 31 >= 128) {
                for (int cb = jw; cb <= (R1 + 32 * q + 31) >> 5; cb += 4) {
                    tmem_ld32(lane_base + 128 + 32 * cb, v);
                    if (r1 >= 128 && r1 < N) {
                        const float nr = nrm[r1];
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const int c = 32 * cb + i;
                            if (c <= r1) d2[r1 * (r1 + 1) / 2 + c] = fmaxf(0.0f, (nr + nrm[c]) - 2.0f * v[i]) * inv_d;
                        }
                    }
                }
            }
        }
        if (dead)  // gave up (flagged): the clustering below still runs, on distances that are all zero, so that
            for (int i = tid; i < L.rows * (L.rows + 1) / 2; i += kMgThreads) d2[i] = 0.0f;  // every index it forms is valid
        tc_fence_before_sync();
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, kMgTmemCols);  // the tensor memory goes back before the clustering starts

        // ================================================================= density peaks: two threads per static token
        // (n_s <= N <= kMgMaxTokens, 2 * kMgMaxTokens <= kMgThreads: thread 2a + h takes the candidates b = h, h + 2, ...
        // of token a; the two are neighbours in a warp and combine by shuffle)
        static_assert(2 * kMgMaxTokens <= kMgThreads, "two threads per token");
        const int kk = min(p.knn, n_s - 1);
        const int a = tid >> 1, hf = tid & 1;
        const bool mine = a < n_s;
        const int ia = mine ? slist[a] : 0, row = ia * (ia + 1) / 2;
        float far2 = 0.0f;  // the token's largest squared distance to another static token
        // KD: slots of the insertion list, at least knn (5, the usual choice, or the maximum of 8)
        auto density = [&](auto kd_tag) {
            constexpr int KD = decltype(kd_tag)::value;
            float best[KD];  // the smallest squared distances among this thread's candidates, ascending
#pragma unroll
            for (int q = 0; q < KD; ++q) best[q] = INFINITY;
            if (mine) {
#pragma unroll 4
                for (int b = hf; b < n_s; b += 2) {
                    const int ib = slist[b];
                    float v = d2[ib <= ia ? row + ib : ib * (ib + 1) / 2 + ia];
                    far2 = fmaxf(far2, v);          // (the token itself adds 0)
                    v = b == a ? INFINITY : v;      // ... and is no neighbour of itself
#pragma unroll
                    for (int q = 0; q < KD; ++q) {  // insertion: v sinks to its place, the largest falls out
                        const float lo = fminf(best[q], v);
                        v = fmaxf(best[q], v);
                        best[q] = lo;
                    }
                }
            }
            // the partner's list sinks into this one: both threads end with the smallest of all candidates
            float theirs[KD];
#pragma unroll
            for (int q = 0; q < KD; ++q) theirs[q] = __shfl_xor_sync(0xffffffffu, best[q], 1);
            far2 = fmaxf(far2, __shfl_xor_sync(0xffffffffu, far2, 1));
#pragma unroll
            for (int e = 0; e < KD; ++e) {
                float v = theirs[e];
#pragma unroll
                for (int q = 0; q < KD; ++q) {
                    const float lo = fminf(best[q], v);
                    v = fmaxf(best[q], v);
                    best[q] = lo;
                }
            }
            float sum = 0.0f;
#pragma unroll
            for (int q = 0; q < KD; ++q)
                if (q < kk) sum += best[q];
            if (mine && hf == 0) rho[a] = kk > 0 ? expf(-sum / (float)kk) : 1.0f;
        };
        if (p.knn <= 5) density(std::integral_constant<int, 5>{});
        else density(std::integral_constant<int, kMgMaxKnn>{});
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
        // the centres in ascending token order: one thread per static token from here on, a warp's share counted by
        // ballot, the warps before it added up (coff is free until the members are sorted)
        const int a1 = tid;
        const int tok1 = a1 < n_s ? slist[a1] : 0;
        {
            const bool is_c = a1 < n_s && flag[tok1] == 3;
            const unsigned bal = __ballot_sync(0xffffffffu, is_c);
            if (lane == 0) coff[warp] = __popc(bal);
            __syncthreads();
            int before = __popc(bal & ((1u << lane) - 1u));
            for (int w = 0; w < warp; ++w) before += coff[w];
            if (is_c) {
                clist[before] = tok1;
                cid[tok1] = before;
            }
        }
        int32_t *wcnt = reinterpret_cast<int32_t *>(smem + L.off_wcnt);
        for (int i = tid; i < (kMgMaxTokens / 32) * L.rows; i += kMgThreads) wcnt[i] = 0;
        __syncthreads();
        // every other static token joins its nearest centre (the earlier centre among equals): the token's two threads
        // take the even and the odd centres
        {
            float bd = INFINITY;
            int best = 0x7fffffff;
            const bool joins = mine && flag[ia] != 3;
            if (joins) {
#pragma unroll 4
                for (int j = hf; j < k_s; j += 2) {
                    const float v = d2[tri(ia, clist[j])];
                    if (v < bd) {
                        bd = v;
                        best = j;
                    }
                }
            }
            const float obd = __shfl_xor_sync(0xffffffffu, bd, 1);
            const int ob = __shfl_xor_sync(0xffffffffu, best, 1);
            if (obd < bd || (obd == bd && ob < best)) best = ob;
            if (joins && hf == 0) cid[ia] = best;
        }
        __syncthreads();
        // members ordered by cluster, ascending token inside a cluster.  A warp holds 32 consecutive static tokens:
        // the lanes of one cluster find each other (match), the first of them records how many they are, and a
        // token's place is its cluster's start + the members in the warps before + those in lower lanes.
        const int c1 = a1 < n_s ? cid[tok1] : -1 - lane;  // (lanes without a token match nobody)
        const unsigned same = __match_any_sync(0xffffffffu, c1);
        if (a1 < n_s && (same & ((1u << lane) - 1u)) == 0) wcnt[warp * L.rows + c1] = __popc(same);
        __syncthreads();
        if (warp == 0) {  // where each cluster starts: a running sum over the clusters, 32 at a time
            int carry = 0;
            for (int j0 = 0; j0 <= k_s; j0 += 32) {
                const int j = j0 + lane;
                int n = 0;
                if (j < k_s)
                    for (int w = 0; w < kMgMaxTokens / 32; ++w) n += wcnt[w * L.rows + j];
                int inc = n;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += v;
                }
                if (j <= k_s) coff[j] = carry + inc - n;
                carry += __shfl_sync(0xffffffffu, inc, 31);
            }
        }
        __syncthreads();
        if (a1 < n_s) {
            int within = __popc(same & ((1u << lane) - 1u));
            for (int w = 0; w < warp; ++w) within += wcnt[w * L.rows + c1];
            member[coff[c1] + within] = tok1;
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
    // a cluster's mean: 8 channels per thread, the members added up in ascending token order.  A thread works on two
    // (cluster, column) items at a time and asks for the first four members of both before it adds any of them up:
    // the rows come from DRAM (they have left L2 since the Gram pass), and what bounds this loop is how many of them
    // are on their way.
    const int n_items = k_s * vec;
    auto first_members = [&](int e, int &j, int &c, int &m0, int &m1, uint4 (&v)[4]) {
        j = e / vec;
        c = e - j * vec;
        m0 = m1 = 0;
        if (e < n_items) {
            m0 = coff[j];
            m1 = coff[j + 1];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            v[u] = m0 + u < m1 ? __ldg(reinterpret_cast<const uint4 *>(Ft + (int64_t)member[m0 + u] * p.st) + c) : make_uint4(0, 0, 0, 0);
    };
    auto add_up = [&](const uint4 (&v)[4], int m, int m1, float (&s8)[8]) {
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
    };
    auto finish = [&](int j, int c, int m0, int m1, uint4 (&v)[4]) {
        float s8[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) s8[q] = 0.0f;
        add_up(v, m0, m1, s8);
        for (int m = m0 + 4; m < m1; m += 4) {  // a cluster of more than four: the rest, four at a time
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = m + u < m1 ? __ldg(reinterpret_cast<const uint4 *>(Ft + (int64_t)member[m + u] * p.st) + c) : make_uint4(0, 0, 0, 0);
            add_up(v, m, m1, s8);
        }
        // The binary32 sum of a few 16-bit values is exact, so a correctly rounded quotient is the correctly rounded
        // mean.  Eight divisions by the same small integer: y = rn(1 / cnt) once, then per value q = rn(s y), the exact
        // remainder r = s - q cnt (one FMA) and q' = rn(q + r y), which is the correctly rounded s / cnt when y is
        // the correctly rounded reciprocal and q is within an ulp (Markstein) -- 3 operations instead of a division.
        const float cnt = (float)(m1 - m0), y = __frcp_rn(cnt);
        float mean[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float q0 = s8[q] * y;
            mean[q] = fmaf(fmaf(-q0, cnt, s8[q]), y, q0);
        }
        uint4 o;
        o.x = pack2<T>(mean[0], mean[1]);
        o.y = pack2<T>(mean[2], mean[3]);
        o.z = pack2<T>(mean[4], mean[5]);
        o.w = pack2<T>(mean[6], mean[7]);
        reinterpret_cast<uint4 *>(ret + (int64_t)slot[j] * D)[c] = o;
    };
    for (int e = tid; e < n_items; e += 2 * kMgThreads) {
        int ja, ca, a0, a1, jb, cb, b0, b1;
        uint4 va[4], vb[4];
        first_members(e, ja, ca, a0, a1, va);
        first_members(e + kMgThreads, jb, cb, b0, b1, vb);
        finish(ja, ca, a0, a1, va);
        if (e + kMgThreads < n_items) finish(jb, cb, b0, b1, vb);
    }
}

}  // namespace stom

using namespace stom;

extern "C" int32_t stom_ctr_merge(const void *F, int32_t dtype, int32_t T, int32_t N, int32_t D, int64_t stride_frame,
                                  int64_t stride_token, const int32_t *k_s, const int32_t *k_d, const int32_t *static_idx,
                                  const int32_t *dyn_idx, int32_t G, int32_t knn, void *retained, int32_t *retained_pos,
                                  int32_t *centre, int32_t *assign, uint32_t *dev_flags, void *stream) {
    if (!F || !k_s || !k_d || !static_idx || !dyn_idx || !retained || !retained_pos || T < 0 || N < 1 || D < 1 || G < 1 || knn < 0)
        return STOM_ERR_INVALID_ARG;
    if (dtype != STOM_BF16 && dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    if (G > N || N > kMgMaxTokens || D % kMgSlabCh || D > 8192 || knn > kMgMaxKnn) return STOM_ERR_SHAPE;
    if (stride_token < D || stride_frame < 0) return STOM_ERR_INVALID_ARG;
    if (!aligned16(F) || !aligned16(retained) || !stride_ok(stride_frame, dtype) || !stride_ok(stride_token, dtype))
        return STOM_ERR_ALIGNMENT;
    const void *ptrs[8] = {k_s, k_d, static_idx, dyn_idx, retained_pos, centre, assign, dev_flags};
    for (const void *q : ptrs)
        if (reinterpret_cast<uintptr_t>(q) & 3u) return STOM_ERR_ALIGNMENT;
    if (T == 0) return STOM_OK;
    MergeParams p{F, stride_frame, stride_token, k_s, k_d, static_idx, dyn_idx, retained, retained_pos, centre, assign, N, D, G, knn, dev_flags};
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
                                          uint32_t *dev_flags, void *stream) {
    // every argument list is checked before the first launch
    if (!retained || !retained_pos || knn < 0) return STOM_ERR_INVALID_ARG;
    if (dtype != STOM_BF16 && dtype != STOM_FP16) return STOM_ERR_UNSUPPORTED;
    if (N < 1 || G < 1 || G > N || N > kMgMaxTokens || D < 1 || D % kMgSlabCh || D > 8192 || knn > kMgMaxKnn) return STOM_ERR_SHAPE;
    if (!aligned16(retained) || (reinterpret_cast<uintptr_t>(retained_pos) & 3u) || (reinterpret_cast<uintptr_t>(dev_flags) & 3u))
        return STOM_ERR_ALIGNMENT;
    int32_t rc = stom_ctr_reduce(F, prev, dtype, T, N, D, stride_frame, stride_token, alpha, G, tau_c, sim, k_s, k_d,
                                 static_idx, dyn_idx, stream);
    if (rc) return rc;
    return stom_ctr_merge(F, dtype, T, N, D, stride_frame, stride_token, k_s, k_d, static_idx, dyn_idx, G, knn, retained,
                          retained_pos, nullptr, nullptr, dev_flags, stream);
}
