// Inline-PTX wrappers (mbarrier, TMA, tcgen05, bit tricks) and the host-side tensor-map encoder
// shared by the sm_100a kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pd_common.cuh"

namespace pd {

constexpr long long kWaitCycles = 2000000000ll;  // ~1 s: far beyond any legitimate wait

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.b32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when the wait ran out or another role of the CTA already gave up;
// the first one to give up latches PD_ERR_DEVICE_TIMEOUT with `where` as detail.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint32_t *status,
                                          uint32_t where, long long limit_cycles = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) {
                *abort_flag = 1;
                latch_error(status, PD_ERR_DEVICE_TIMEOUT, where);
                return false;
            }
        }
    }
}

// ------------------------------------------------------------------ TMA
__device__ __forceinline__ void tma_load_2d(const CUtensorMap *map, uint64_t *bar, void *dst, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(const CUtensorMap *map, uint64_t *bar, void *dst, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
// untiled copy: both addresses 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ------------------------------------------------------------------ bit tricks
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// (~a & b) | c
__device__ __forceinline__ uint32_t lop3_andn_or(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xAE;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// (~a & b) ^ c
__device__ __forceinline__ uint32_t lop3_andn_xor(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xA6;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t hadd2_u32(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// ------------------------------------------------------------------ the two storage types of weights and activations
// Elem<false>: IEEE binary16; Elem<true>: bfloat16 (paper, Implementation remarks: the base is kept in BF16).  Values
// travel as raw bits (one element per unsigned short, two per 32-bit register, the lower index in the lower half).
// The scale vectors are binary16 in both cases.
template <bool BF16>
struct Elem;

template <>
struct Elem<false> {
    static constexpr uint32_t kOnePair = 0x3C003C00u;  // (1.0, 1.0)
    static __device__ __forceinline__ float to_float(unsigned short h) { return __half2float(__ushort_as_half(h)); }
    static __device__ __forceinline__ float2 to_float2(uint32_t p) { return __half22float2(*reinterpret_cast<const __half2 *>(&p)); }
    static __device__ __forceinline__ unsigned short from_float(float f) { return __half_as_ushort(__float2half_rn(f)); }
    static __device__ __forceinline__ uint32_t from_float2(float lo, float hi) {
        const __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t *>(&h);
    }
    static __device__ __forceinline__ uint32_t add2(uint32_t a, uint32_t b) { return hadd2_u32(a, b); }
    // 0xffff in every half where a >= b (false for NaN, true for -0 against +0)
    static __device__ __forceinline__ uint32_t ge_mask(uint32_t a, uint32_t b) {
        return __hge2_mask(*reinterpret_cast<const __half2 *>(&a), *reinterpret_cast<const __half2 *>(&b));
    }
    // a binary16 scale as a pair (s, s) of elements, and a pair of binary16 scales as a pair of elements
    static __device__ __forceinline__ uint32_t scale_pair(unsigned short v) { return static_cast<uint32_t>(v) | (static_cast<uint32_t>(v) << 16); }
    static __device__ __forceinline__ uint32_t scale_pair2(uint32_t v2) { return v2; }
    static __device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};

template <>
struct Elem<true> {
    static constexpr uint32_t kOnePair = 0x3F803F80u;
    static __device__ __forceinline__ float to_float(unsigned short h) { return __uint_as_float(static_cast<uint32_t>(h) << 16); }
    static __device__ __forceinline__ float2 to_float2(uint32_t p) { return make_float2(__uint_as_float(p << 16), __uint_as_float(p & 0xffff0000u)); }
    static __device__ __forceinline__ unsigned short from_float(float f) { return __bfloat16_as_ushort(__float2bfloat16_rn(f)); }
    static __device__ __forceinline__ uint32_t from_float2(float lo, float hi) {
        uint32_t d;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
        return d;
    }
    static __device__ __forceinline__ uint32_t add2(uint32_t a, uint32_t b) {
        uint32_t d;
        asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
        return d;
    }
    static __device__ __forceinline__ uint32_t ge_mask(uint32_t a, uint32_t b) {
        return __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
    }
    // the scale is rounded to bfloat16 once, to nearest even
    static __device__ __forceinline__ uint32_t scale_pair(unsigned short v) {
        const uint32_t b = from_float(__half2float(__ushort_as_half(v)));
        return b | (b << 16);
    }
    static __device__ __forceinline__ uint32_t scale_pair2(uint32_t v2) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&v2));
        return from_float2(f.x, f.y);
    }
    static __device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};

// ------------------------------------------------------------------ host: tensor maps
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Row-major 2-D tensor [rows, cols] with row pitch `pitch_bytes` (a multiple of 16); box = box_cols x box_rows
// elements; out-of-range elements read as zero.
inline bool make_map_2d(CUtensorMap *map, CUtensorMapDataType type, int elem_bytes, const void *base, int64_t rows,
                        int64_t cols, int64_t pitch_bytes, int box_cols, int box_rows, CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    (void)elem_bytes;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch_bytes)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, type, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-major fp16 matrix [rows, cols] (cols a multiple of 64, row pitch a multiple of 128 bytes) seen as
// {64 columns, cols/64 column blocks, rows}: one box of {64, blocks, box_rows} brings `blocks` swizzled
// 128-byte pieces of each of box_rows rows with a single instruction.  In shared memory a row of the box
// is blocks*128 contiguous bytes; the 16-byte piece index is XORed with bits 7..9 of the byte offset.
inline bool make_map_blocked_f16(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t pitch_bytes,
                                 int blocks, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(cols / 64), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[2] = {128, static_cast<cuuint64_t>(pitch_bytes)};
    const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(blocks), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Packed mask [rows, cols/32 words] (cols a multiple of 128) seen as {4 words, rows, cols/128 groups}: one box of
// {4, box_rows, box_groups} lands in shared memory as [group][row][4 words], i.e. the 16 bytes of consecutive
// rows are adjacent.  Groups past the end read as zeros.
inline bool make_map_mask_groups(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int box_rows,
                                 int box_groups) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {4, static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(cols / 128)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(cols / 8), 16};
    const cuuint32_t box[3] = {4, static_cast<cuuint32_t>(box_rows), static_cast<cuuint32_t>(box_groups)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace pd
