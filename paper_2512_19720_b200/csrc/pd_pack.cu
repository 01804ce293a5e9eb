// pack: sign mask of W_f - W_b plus the exact per-axis sums of |W_f - W_b|, and
// merge: W_hat = fp16(fp32(W_b) +- fp32(v)).  Both are single-pass streaming kernels bound by HBM
// (4.125 bytes per weight element each).
//
// Tile shape for both: a CTA of 8 warps covers 64 rows x 256 columns; a warp owns one row at a
// time, a lane owns 8 consecutive columns (one 128-bit load per matrix), so four neighbouring
// lanes form one 32-bit mask word.
#include "pd_common.cuh"

namespace pd {

std::atomic<int64_t> g_launches{0};

namespace {

constexpr int kThreads = 256;
constexpr int kTileRows = 64;
constexpr int kTileCols = 256;
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// same without the read-only path: merge may write its output over its input
__device__ __forceinline__ uint4 ldg_stream_coherent(const uint4 *p) {
    uint4 r;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p)
                 : "memory");
    return r;
}

__device__ __forceinline__ void stg_stream(uint4 *p, uint4 v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

__device__ __forceinline__ __half2 as_half2(uint32_t u) { return *reinterpret_cast<__half2 *>(&u); }

// Signed value of a binary16 in units of 2^-24 (every finite binary16 is an integer number of them).
__device__ __forceinline__ long long half_units(uint32_t h) {
    const uint32_t e = (h >> 10) & 31u, m = h & 1023u;
    const long long mag = e ? (static_cast<long long>(m | 1024u) << (e - 1u)) : static_cast<long long>(m);
    return (h & 0x8000u) ? -mag : mag;
}

// |a - b| in units of 2^-24 for two binary16 values less than 0.5 apart: the fp32 difference is exact
// (a multiple of 2^-24 below 2^23 units), and adding 0.5 places it where one fp32 ulp is 2^-24.  For
// values 0.5 or more apart the result is >= 2^23 (or has high bits set), which the caller tests.
__device__ __forceinline__ uint32_t abs_diff_units_small(float a, float b) {
    return __float_as_uint(fabsf(__fsub_rn(a, b)) + 0.5f) - 0x3f000000u;
}

// Programmatic dependent launch: a pack call is three kernels (zero the sums, pack, finalize).  Each lets the
// next one be scheduled as soon as it has started and the next one waits for it before it touches the sums, so
// the launch latencies overlap the kernels instead of adding to them.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__global__ void zero_sums_kernel(unsigned long long *__restrict__ sums, int n) {
    grid_launch_dependents();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) sums[i] = 0ull;
}

template <bool ROW, bool COL>
__global__ void __launch_bounds__(kThreads)
pack_kernel(const uint4 *__restrict__ w_f, const uint4 *__restrict__ w_b, int d_out, int d_in, int tiles_c,
            uint32_t *__restrict__ mask, unsigned long long *__restrict__ row_sum,
            unsigned long long *__restrict__ col_sum) {
    __shared__ uint32_t s_col[COL ? (kThreads / 32) * kTileCols : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tile_r = blockIdx.x / tiles_c, tile_c = blockIdx.x - tile_r * tiles_c;
    const int col0 = tile_c * kTileCols + lane * 8;
    const int row0 = tile_r * kTileRows;
    const bool col_ok = col0 < d_in;
    const int words = d_in >> 5;

    uint32_t cacc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) cacc[j] = 0;
    grid_launch_dependents();  // the finalize kernel may be scheduled; it waits for this grid

#pragma unroll 4
    for (int rr = warp; rr < kTileRows; rr += kThreads / 32) {
        const int o = row0 + rr;
        if (o >= d_out) break;  // warp-uniform
        uint32_t bits = 0, fast_sum = 0;
        unsigned long long slow_sum = 0;
        bool slow = false;
        uint4 a4 = make_uint4(0, 0, 0, 0), b4 = a4;
        if (col_ok) {
            const size_t idx = (static_cast<size_t>(o) * d_in + col0) >> 3;
            a4 = ldg_stream(w_f + idx), b4 = ldg_stream(w_b + idx);
        }
        // the first loads are in flight; nothing may be added to the sums before the kernel that zeroes them is done
        if (rr == warp) grid_dependency_wait();
        if (col_ok) {
            const uint32_t a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
            uint32_t spread = 0, u[8], u_or = 0;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                // bit = (w_f >= w_b): exact on binary16, false for NaN, true for -0 vs +0.  The comparison gives
                // 0xffff per true half; pair p keeps bit 2p of the low half and bit 2p+1 of the high half.
                const uint32_t ge = __hge2_mask(as_half2(a[p]), as_half2(b[p]));
                spread |= ge & ((1u << (2 * p)) | (1u << (17 + 2 * p)));
                // |dW| in units of 2^-24 by the fp32 trick.  Every binary16 is a multiple of 2^-24, so whenever
                // |dW| < 0.5 the fp32 difference is exact and |dW| + 0.5 lies in [0.5, 1), where one ulp is 2^-24.
                const float2 fa = __half22float2(as_half2(a[p])), fb = __half22float2(as_half2(b[p]));
                u[2 * p] = abs_diff_units_small(fa.x, fb.x);
                u[2 * p + 1] = abs_diff_units_small(fa.y, fb.y);
                u_or |= u[2 * p] | u[2 * p + 1];
            }
            bits = (spread | (spread >> 16)) & 0xffu;
            slow = (u_or & 0xff800000u) != 0;  // some |dW| >= 0.5 (or not finite): take the exact 64-bit path
            if (!slow) {
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    if (COL) {
                        cacc[2 * p] += u[2 * p];
                        cacc[2 * p + 1] += u[2 * p + 1];
                    }
                    fast_sum += u[2 * p] + u[2 * p + 1];
                }
            } else {
#pragma unroll
                for (int p = 0; p < 4; ++p) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const long long d = half_units((a[p] >> (16 * h)) & 0xffffu) -
                                            half_units((b[p] >> (16 * h)) & 0xffffu);
                        const unsigned long long du = static_cast<unsigned long long>(d < 0 ? -d : d);
                        slow_sum += du;
                        if (COL) atomicAdd(col_sum + col0 + 2 * p + h, du);
                    }
                }
            }
        }
        uint32_t word = bits << (8 * (lane & 3));
        word |= __shfl_xor_sync(kFull, word, 1);
        word |= __shfl_xor_sync(kFull, word, 2);
        if ((lane & 3) == 0 && col_ok) mask[static_cast<size_t>(o) * words + (col0 >> 5)] = word;
        if (ROW) {
            // each lane adds at most 8 * 2^23 units on the fast path, so the 32-lane sum fits 32 bits
            unsigned long long total = __reduce_add_sync(kFull, fast_sum);
            if (__any_sync(kFull, slow)) {
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) slow_sum += __shfl_xor_sync(kFull, slow_sum, s);
                total += slow_sum;
            }
            if (lane == 0) atomicAdd(row_sum + o, total);
        }
    }
    grid_dependency_wait();  // warps without a row in this tile have not waited yet
    if (COL) {
#pragma unroll
        for (int j = 0; j < 8; ++j) s_col[warp * kTileCols + lane * 8 + j] = cacc[j];
        __syncthreads();
        const int c = tile_c * kTileCols + threadIdx.x;
        if (c < d_in) {
            uint32_t t = 0;  // <= 64 rows * 2^23 units
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) t += s_col[w * kTileCols + threadIdx.x];
            atomicAdd(col_sum + c, static_cast<unsigned long long>(t));
        }
    }
}

// mean = (sum * 2^-24) / n with one fp64 division, then one rounding to binary16
__global__ void pack_finalize_kernel(const unsigned long long *__restrict__ row_sum,
                                     const unsigned long long *__restrict__ col_sum, int d_out, int d_in,
                                     __half *__restrict__ v_row, __half *__restrict__ v_col) {
    grid_dependency_wait();  // every tile has added its sums
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const bool is_row = idx < d_out;
    const int j = is_row ? idx : idx - d_out;
    if (!is_row && j >= d_in) return;
    __half *dst = is_row ? v_row : v_col;
    if (dst == nullptr) return;
    const unsigned long long s = is_row ? row_sum[j] : col_sum[j];
    const double q = __ddiv_rn(static_cast<double>(s), static_cast<double>(is_row ? d_in : d_out)) *
                     5.9604644775390625e-08;  // 2^-24, exact scaling
    unsigned short h;
    asm("cvt.rn.f16.f64 %0, %1;" : "=h"(h) : "d"(q));
    reinterpret_cast<unsigned short *>(dst)[j] = h;
}

template <int AXIS>
__global__ void __launch_bounds__(kThreads)
merge_kernel(const uint4 *w_b, const uint32_t *__restrict__ mask, const __half *__restrict__ v, int d_out, int d_in,
             int tiles_c, uint4 *w_hat) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tile_r = blockIdx.x / tiles_c, tile_c = blockIdx.x - tile_r * tiles_c;
    const int col0 = tile_c * kTileCols + lane * 8;
    const int row0 = tile_r * kTileRows;
    if (col0 >= d_in) return;
    const int words = d_in >> 5;
    float vf[8];
    if (AXIS == PD_AXIS_COL) {
        const uint4 vv = *reinterpret_cast<const uint4 *>(v + col0);
        const uint32_t u[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const float2 f = __half22float2(as_half2(u[p]));
            vf[2 * p] = f.x;
            vf[2 * p + 1] = f.y;
        }
    }
#pragma unroll 8
    for (int rr = warp; rr < kTileRows; rr += kThreads / 32) {
        const int o = row0 + rr;
        if (o >= d_out) break;
        const size_t idx = (static_cast<size_t>(o) * d_in + col0) >> 3;
        const uint4 w4 = ldg_stream_coherent(w_b + idx);
        const uint32_t word = __ldg(mask + static_cast<size_t>(o) * words + (col0 >> 5));
        const uint32_t nbits = ~(word >> (8 * (lane & 3)));  // bit set -> B = -1
        if (AXIS == PD_AXIS_ROW) {
            const float s = __half2float(v[o]);
#pragma unroll
            for (int j = 0; j < 8; ++j) vf[j] = s;
        }
        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
        uint32_t r[4];
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const float2 f = __half22float2(as_half2(w[p]));
            const float s0 = __uint_as_float(__float_as_uint(vf[2 * p]) ^ (((nbits >> (2 * p)) & 1u) << 31));
            const float s1 = __uint_as_float(__float_as_uint(vf[2 * p + 1]) ^ (((nbits >> (2 * p + 1)) & 1u) << 31));
            const __half2 h = __floats2half2_rn(__fadd_rn(f.x, s0), __fadd_rn(f.y, s1));
            r[p] = *reinterpret_cast<const uint32_t *>(&h);
        }
        stg_stream(w_hat + idx, make_uint4(r[0], r[1], r[2], r[3]));
    }
}

}  // namespace

pd_status launch_pack(const __half *w_f, const __half *w_b, int64_t d_out, int64_t d_in, uint32_t *mask,
                      __half *v_row, __half *v_col, unsigned long long *sums, cudaStream_t stream) {
    unsigned long long *row_sum = sums, *col_sum = sums + d_out;
    const int n = static_cast<int>(d_out + d_in);
    zero_sums_kernel<<<(n + 255) / 256, 256, 0, stream>>>(sums, n);
    const int tiles_c = static_cast<int>((d_in + kTileCols - 1) / kTileCols);
    const int64_t tiles = ((d_out + kTileRows - 1) / kTileRows) * tiles_c;
    const uint4 *a = reinterpret_cast<const uint4 *>(w_f), *b = reinterpret_cast<const uint4 *>(w_b);
    const int n_out = static_cast<int>(d_out), n_in = static_cast<int>(d_in);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may be scheduled while the previous kernel runs
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(tiles));
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (v_row && v_col)
        e = cudaLaunchKernelEx(&cfg, pack_kernel<true, true>, a, b, n_out, n_in, tiles_c, mask, row_sum, col_sum);
    else if (v_row)
        e = cudaLaunchKernelEx(&cfg, pack_kernel<true, false>, a, b, n_out, n_in, tiles_c, mask, row_sum, col_sum);
    else
        e = cudaLaunchKernelEx(&cfg, pack_kernel<false, true>, a, b, n_out, n_in, tiles_c, mask, row_sum, col_sum);
    if (e != cudaSuccess) return PD_ERR_CUDA;
    cfg.gridDim = dim3(static_cast<unsigned>((n + 255) / 256));
    cfg.blockDim = dim3(256);
    if (cudaLaunchKernelEx(&cfg, pack_finalize_kernel, static_cast<const unsigned long long *>(row_sum),
                           static_cast<const unsigned long long *>(col_sum), n_out, n_in, v_row, v_col) != cudaSuccess)
        return PD_ERR_CUDA;
    count_launch(3);
    return cuda_ok(cudaGetLastError());
}

pd_status launch_merge(const __half *w_b, const uint32_t *mask, const __half *v, int axis, int64_t d_out,
                       int64_t d_in, __half *w_hat, cudaStream_t stream) {
    const int tiles_c = static_cast<int>((d_in + kTileCols - 1) / kTileCols);
    const int64_t tiles = ((d_out + kTileRows - 1) / kTileRows) * tiles_c;
    const dim3 grid(static_cast<unsigned>(tiles)), block(kThreads);
    const uint4 *b = reinterpret_cast<const uint4 *>(w_b);
    uint4 *out = reinterpret_cast<uint4 *>(w_hat);
    if (axis == PD_AXIS_ROW)
        merge_kernel<PD_AXIS_ROW><<<grid, block, 0, stream>>>(b, mask, v, (int)d_out, (int)d_in, tiles_c, out);
    else
        merge_kernel<PD_AXIS_COL><<<grid, block, 0, stream>>>(b, mask, v, (int)d_out, (int)d_in, tiles_c, out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace pd

// ---------------------------------------------------------------------------------------------
// pd_pack_delta_static: the pack call for callers that cannot hand over a workspace.
//
// The exact sums of |dW| (one 64-bit word per output row and per input column) live in the
// file-scope device array below instead of in caller memory.  The array is part of the loaded
// module: every GPU that loads the library carries its 512 KiB until the process exits.
// In host code `g_static_sums` is only a handle; the device address comes from
// cudaGetSymbolAddress, asked once per device with that device current.
namespace pd {
namespace {

constexpr int64_t kStaticSumWords = 65536;  // d_out + d_in may not exceed this
static __device__ __align__(256) unsigned long long g_static_sums[kStaticSumWords];

std::atomic<unsigned long long *> g_static_sums_addr[kMaxDevices];

// Device address of g_static_sums on the current device (nullptr on failure).
unsigned long long *static_sums_on_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    unsigned long long *p = g_static_sums_addr[dev].load(std::memory_order_acquire);
    if (p != nullptr) return p;
    void *sym = nullptr;
    if (cudaGetSymbolAddress(&sym, g_static_sums) != cudaSuccess || sym == nullptr) return nullptr;
    p = static_cast<unsigned long long *>(sym);
    g_static_sums_addr[dev].store(p, std::memory_order_release);  // every thread resolves the same address
    return p;
}

}  // namespace
}  // namespace pd

extern "C" pd_status pd_pack_delta_static(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in,
                                          uint32_t *mask, void *v_row, void *v_col, void *cuda_stream) {
    using namespace pd;
    if (!w_f || !w_b || !mask || (!v_row && !v_col) || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    if (d_in % 32 != 0 || d_out > kStaticSumWords || d_in > kStaticSumWords || d_out + d_in > kStaticSumWords)
        return PD_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(w_f) || !aligned16(w_b) || (reinterpret_cast<uintptr_t>(mask) & 3u)) return PD_ERR_ALIGNMENT;
    unsigned long long *sums = static_sums_on_current_device();
    if (sums == nullptr) return PD_ERR_CUDA;
    // launch_pack zero-fills sums[0 .. d_out + d_in) on the stream before the kernel adds into it
    return launch_pack(static_cast<const __half *>(w_f), static_cast<const __half *>(w_b), d_out, d_in, mask,
                       static_cast<__half *>(v_row), static_cast<__half *>(v_col), sums,
                       static_cast<cudaStream_t>(cuda_stream));
}
