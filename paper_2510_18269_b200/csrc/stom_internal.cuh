// Internal helpers shared by the translation units of libstom_oqm.so.
// Host side: argument validation, bank addressing, CUDA error bookkeeping.
// Device side: vector loads and number-format helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "stom_oqm.h"

namespace stom {

// ---------------------------------------------------------------- host

void set_last_cuda_error(cudaError_t e);

// Validates the geometry; returns STOM_OK or an error code.
int32_t check_config(const stom_oqm_config *cfg);
int32_t check_store(const stom_oqm_store *st);
int32_t check_layers(const stom_oqm_config *cfg, int32_t layer_begin, int32_t layer_count);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int elem_bytes(int dtype) { return dtype == STOM_FP32 ? 4 : 2; }
inline bool stride_ok(int64_t stride_elems, int dtype) { return (stride_elems * elem_bytes(dtype)) % 16 == 0; }

inline int32_t finish_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_last_cuda_error(e);
        return STOM_ERR_CUDA;
    }
    return STOM_OK;
}

// Bank geometry passed by value to kernels.
struct BankGeom {
    int32_t H;        // kv heads
    int32_t G;        // tokens per group
    int32_t d;        // head dim
    int32_t cap;      // groups per layer
    int32_t row_bytes;  // packed bytes per token row = d * bits / 8
    int32_t meta_dtype;  // STOM_FP32 | STOM_FP16 | STOM_BF16: element type of the s, m and k-bar arrays
};

inline BankGeom bank_geom(const stom_oqm_config *c) {
    return BankGeom{c->n_kv_heads, c->group_tokens, c->head_dim, c->capacity_groups, c->head_dim * c->bits / 8,
                    c->meta_dtype};
}

// A2+A3 -> A4 inside one retrieval: same checks and launch as stom_oqm_dequant_gather; `after_producer` launches the
// kernel with programmatic stream serialization, so that its blocks may be scheduled while the kernel ahead of it in
// the stream (which wrote idx) is still draining -- the kernel itself waits for that grid before it reads idx.
int32_t dequant_gather_launch(const stom_oqm_config *cfg, const stom_oqm_store *store, int32_t layer_begin,
                              int32_t layer_count, const int32_t *idx, int32_t k, int32_t n_groups, void *k_active,
                              void *v_active, int32_t out_dtype, int64_t stride_layer, int64_t stride_head,
                              int64_t stride_token, int32_t token_offset, uint32_t *dev_flags, void *stream,
                              bool after_producer);

// ---------------------------------------------------------------- device

#ifdef __CUDACC__

// Programmatic dependent launch (sm_90+).  grid_dependency_wait: returns once the grids this one depends on have
// completed and their writes are visible (at once if the launch had no programmatic dependency).
// grid_launch_dependents: lets a dependent grid start being scheduled from here on.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launches `kernel` so that it may overlap the tail of the kernel ahead of it in the stream.
template <typename P>
inline cudaError_t launch_after_producer(void (*kernel)(P), dim3 grid, dim3 block, size_t smem, cudaStream_t s, const P &p) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kernel, p);
}

// Index of (layer, group, head) in the [L][cap][H] lattice every bank array shares.
__device__ __forceinline__ int64_t bank_slot(const BankGeom &g, int l, int t, int h) {
    return ((int64_t)l * g.cap + t) * g.H + h;
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Two packed 16-bit elements -> two floats (exact).
template <typename T>
__device__ __forceinline__ void unpack2(uint32_t w, float &a, float &b);
template <>
__device__ __forceinline__ void unpack2<__nv_bfloat16>(uint32_t w, float &a, float &b) {
    a = bf16lo(w);
    b = bf16hi(w);
}
template <>
__device__ __forceinline__ void unpack2<__half>(uint32_t w, float &a, float &b) {
    __half2 h = *reinterpret_cast<__half2 *>(&w);
    float2 f = __half22float2(h);
    a = f.x;
    b = f.y;
}

// Two floats -> two packed 16-bit elements, round to nearest even.
template <typename T>
__device__ __forceinline__ uint32_t pack2(float a, float b);
template <>
__device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}
template <>
__device__ __forceinline__ uint32_t pack2<__half>(float a, float b) {
    __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Eight adjacent values of a bank array of s, m or k-bar (element type MT), starting at element `at` (a multiple of
// 8), as floats.
template <typename MT>
__device__ __forceinline__ void load_meta8(const void *base, int64_t at, float (&f)[8]) {
    if constexpr (sizeof(MT) == 4) {
        const float4 *p = reinterpret_cast<const float4 *>(static_cast<const float *>(base) + at);
        const float4 a = __ldg(p), b = __ldg(p + 1);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    } else {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(static_cast<const MT *>(base) + at));
        unpack2<MT>(v.x, f[0], f[1]);
        unpack2<MT>(v.y, f[2], f[3]);
        unpack2<MT>(v.z, f[4], f[5]);
        unpack2<MT>(v.w, f[6], f[7]);
    }
}

// A (scale, offset) pair of 8 channels with the element type known only at run time: one warp-uniform branch around
// both loads, so that they are in flight together.  Used where the load happens once per unit of work.
__device__ __forceinline__ void load_scale_zero8(const void *scale, const void *zero, int64_t at, int meta_dtype,
                                                 float (&s)[8], float (&m)[8]) {
    if (meta_dtype == STOM_FP32) {
        load_meta8<float>(scale, at, s);
        load_meta8<float>(zero, at, m);
    } else if (meta_dtype == STOM_BF16) {
        load_meta8<__nv_bfloat16>(scale, at, s);
        load_meta8<__nv_bfloat16>(zero, at, m);
    } else {
        load_meta8<__half>(scale, at, s);
        load_meta8<__half>(zero, at, m);
    }
}

// The codes of 8 adjacent channels (32 bits at 4 bits per code, 16 bits at 2), each as the bit pattern of the float
// 2^23 + code: a byte permute drops the code into the low mantissa byte of 0x4B000000, so that subtracting 2^23
// leaves the integer without a conversion instruction.  Channel c sits in bits [BITS*c, BITS*c + BITS).
template <int BITS>
__device__ __forceinline__ void code_floats8(uint32_t w, uint32_t (&f)[8]) {
    if constexpr (BITS == 4) {
        const uint32_t even = w & 0x0f0f0f0fu;        // byte i: code of channel 2i
        const uint32_t odd = (w >> 4) & 0x0f0f0f0fu;  // byte i: code of channel 2i+1
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __byte_perm(even, 0x4B000000u, 0x7540u + i);
            f[2 * i + 1] = __byte_perm(odd, 0x4B000000u, 0x7540u + i);
        }
    } else {
        uint32_t t[4];  // t[j], byte b: code of channel 4b + j
#pragma unroll
        for (int j = 0; j < 4; ++j) t[j] = (w >> (2 * j)) & 0x0303u;
#pragma unroll
        for (int c = 0; c < 8; ++c) f[c] = __byte_perm(t[c & 3], 0x4B000000u, 0x7540u + (c >> 2));
    }
}

// The packed codes of 8 adjacent channels of one row: p points at the row, cl is the 8-channel block.
template <int BITS>
__device__ __forceinline__ uint32_t load_codes8(const uint8_t *row, int cl) {
    if constexpr (BITS == 4) return __ldg(reinterpret_cast<const uint32_t *>(row) + cl);
    else return __ldg(reinterpret_cast<const uint16_t *>(row) + cl);
}

// W consecutive 32-bit words from global memory through the read-only path.
template <int W>
struct Words {
    uint32_t w[W];
};

template <int W>
__device__ __forceinline__ Words<W> load_words(const void *p) {
    Words<W> r;
    if constexpr (W == 1) {
        r.w[0] = __ldg(reinterpret_cast<const uint32_t *>(p));
    } else if constexpr (W == 2) {
        uint2 v = __ldg(reinterpret_cast<const uint2 *>(p));
        r.w[0] = v.x;
        r.w[1] = v.y;
    } else {
        static_assert(W % 4 == 0, "word count");
#pragma unroll
        for (int i = 0; i < W / 4; ++i) {
            uint4 v = __ldg(reinterpret_cast<const uint4 *>(p) + i);
            r.w[4 * i + 0] = v.x;
            r.w[4 * i + 1] = v.y;
            r.w[4 * i + 2] = v.z;
            r.w[4 * i + 3] = v.w;
        }
    }
    return r;
}

// Element j of a register-resident row fragment as float.
template <typename T, int W>
__device__ __forceinline__ float elem_of(const Words<W> &r, int j) {
    if constexpr (sizeof(T) == 4) {
        return __uint_as_float(r.w[j]);
    } else {
        float a, b;
        unpack2<T>(r.w[j >> 1], a, b);
        return (j & 1) ? b : a;
    }
}

#endif  // __CUDACC__

}  // namespace stom
