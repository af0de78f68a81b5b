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
#include "stom_topk.cuh"

using namespace stom;

extern "C" int32_t stom_oqm_topk(const float *scores, int32_t rows, int32_t n, int64_t row_stride, int32_t k,
                                 int32_t *idx_out, float *score_out, int32_t *n_sel_out, void *stream) {
    if (!scores || !idx_out || rows < 0 || n < 0 || k < 1 || row_stride < n) return STOM_ERR_INVALID_ARG;
    if (n > (1 << 24)) return STOM_ERR_SHAPE;
    if (rows == 0) return STOM_OK;
    TopkParams p{scores, row_stride, n, k, idx_out, score_out, n_sel_out};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n <= kTopkRegKeys * kTopkBlock) {
        topk_kernel<kKeysRegs><<<rows, kTopkBlock, 0, s>>>(p);
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
        topk_kernel<kKeysShared><<<rows, kTopkBlock, smem, s>>>(p);
    } else {
        topk_kernel<kKeysGlobal><<<rows, kTopkBlock, 0, s>>>(p);
    }
    return finish_launch();
}
