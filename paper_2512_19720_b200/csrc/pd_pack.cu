// pack: sign mask of W_f - W_b plus the exact per-axis means of |W_f - W_b|, and
// merge: W_hat = fp16(fp32(W_b) +- fp32(v)).  Both are single-pass streaming kernels bound by HBM
// (4.125 bytes per weight element each).
//
// Tile shape: a CTA of 8 warps covers 32 (pack) or 64 (merge) rows x 256 columns; a warp owns one row at a
// time, a lane owns 8 consecutive columns (one 128-bit load per matrix), so four neighbouring
// lanes form one 32-bit mask word.
#include <climits>

#include "pd_ptx.cuh"

namespace pd {

std::atomic<int64_t> g_launches{0};

namespace {

constexpr int kThreads = 256;
constexpr int kTileRows = 64;   // merge
constexpr int kPackRows = 32;   // pack
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

// floor(|a - b| * 2^24) for two finite values of at most 2^28 in magnitude: the fp64 difference is taken with
// rounding toward zero, which cuts |a - b| down to a grid finer than 2^-24 and so never crosses a multiple of
// 2^-24; the product with 2^24 is exact and the conversion rounds down.  (binary16 differences are multiples of
// 2^-24 already: nothing is cut.)
__device__ __forceinline__ unsigned long long abs_diff_units(float a, float b) {
    const double d = fabs(__dsub_rz(static_cast<double>(a), static_cast<double>(b)));
    return __double2ull_rd(d * 16777216.0);
}

// mean = (sum * 2^-24) / n with one fp64 division, then one rounding to binary16
__device__ __forceinline__ unsigned short mean_to_half(unsigned long long sum, int n) {
    const double q = __ddiv_rn(static_cast<double>(sum), static_cast<double>(n)) * 5.9604644775390625e-08;  // 2^-24, exact scaling
    unsigned short h;
    asm("cvt.rn.f16.f64 %0, %1;" : "=h"(h) : "d"(q));
    return h;
}

// One row of a tile, any position: bounds-checked, exact 64-bit fixed point for every magnitude.  Used for tiles that
// hang over the matrix edge and for the rare tiles that hold a |dW| >= 0.5.
template <bool BF16, bool ROW, bool COL>
__device__ __forceinline__ void pack_row_exact(const uint4 *__restrict__ w_f, const uint4 *__restrict__ w_b, int o, int col0,
                                               int d_out, int d_in, uint32_t *__restrict__ mask,
                                               unsigned long long *__restrict__ row_sum,
                                               unsigned long long *__restrict__ col_sum, int lane) {
    const bool ok = o < d_out && col0 < d_in;
    uint32_t bits = 0;
    unsigned long long sum = 0;
    if (ok) {
        const size_t idx = (static_cast<size_t>(o) * d_in + col0) >> 3;
        const uint4 a4 = ldg_stream(w_f + idx), b4 = ldg_stream(w_b + idx);
        const uint32_t a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const uint32_t ge = Elem<BF16>::ge_mask(a[p], b[p]);
            bits |= ((ge & 1u) << (2 * p)) | (((ge >> 16) & 1u) << (2 * p + 1));
            const float2 fa = Elem<BF16>::to_float2(a[p]), fb = Elem<BF16>::to_float2(b[p]);
            const unsigned long long du[2] = {abs_diff_units(fa.x, fb.x), abs_diff_units(fa.y, fb.y)};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                sum += du[h];
                if (COL) atomicAdd(col_sum + col0 + 2 * p + h, du[h]);
            }
        }
    }
    uint32_t word = bits << (8 * (lane & 3));
    word |= __shfl_xor_sync(kFull, word, 1);
    word |= __shfl_xor_sync(kFull, word, 2);
    if ((lane & 3) == 0 && ok) mask[static_cast<size_t>(o) * (d_in >> 5) + (col0 >> 5)] = word;
    if (ROW) {
#pragma unroll
        for (int sft = 16; sft > 0; sft >>= 1) sum += __shfl_xor_sync(kFull, sum, sft);
        if (lane == 0 && o < d_out) atomicAdd(row_sum + o, sum);
    }
}

// Programmatic dependent launch: a pack call is two kernels (pack, then the small kernel that turns sums into
// scales).  The first lets the second be scheduled as soon as it has started and the second waits for it before it
// touches the sums, so the second launch's latency overlaps the first kernel.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// A CTA of 8 warps packs one tile of 32 rows x 256 columns; warp w owns rows w, w + 8, w + 16, w + 24, a lane 8
// consecutive columns.  All eight 16-byte loads of a thread (4 rows x 2 matrices) are issued before any arithmetic,
// a CTA makes a single round trip to memory, and four CTAs share an SM, so that one CTA's arithmetic overlaps the
// others' loads.  (Measured and dropped: 64-row tiles with sixteen loads per thread -- half the occupancy; persistent
// CTAs that prefetch their next tile, and one tile per warp with double-buffered batches -- several dependent round
// trips per thread, which a 20 us kernel cannot hide; finishing a band in the CTA that draws its last ticket instead
// of in a second kernel -- the fence and the ticket's round trip hold the whole CTA for longer than its loads take.)
//
// What is summed is floor(|dW| * 2^24) units of 2^-24, exactly (for binary16 inputs |dW| is a whole number of them).
// The fp32 difference rounded toward zero is |dW| cut down to a grid finer than 2^-24 (exact for binary16); an fp32
// accumulator that starts at 0.5 and stays below 1 has an ulp of 2^-24, so adding |dW| to it with rounding toward
// zero adds exactly the whole units of |dW|, and its bit pattern minus that of 0.5 is the sum in units.  A lane keeps
// one such accumulator per row (8 addends) and one per column (4 addends).  An accumulator that reaches 1 (or is
// not finite) fails the check and that row, or that warp's share of the columns, is redone by pack_row_exact in
// 64-bit integers; so are tiles that hang over the matrix edge.
template <bool BF16, bool ROW, bool COL>
__global__ void __launch_bounds__(kThreads, 4)
pack_kernel(const uint4 *__restrict__ w_f, const uint4 *__restrict__ w_b, int d_out, int d_in, int tiles_c,
            uint32_t *__restrict__ mask, unsigned long long *__restrict__ row_sum,
            unsigned long long *__restrict__ col_sum) {
    __shared__ uint32_t s_col[COL ? (kThreads / 32) * kTileCols : 1];
    constexpr int kRowsPerWarp = kPackRows / (kThreads / 32);  // 4
    constexpr uint32_t kHalfBits = 0x3f000000u, kOneBits = 0x3f800000u;  // bit patterns of 0.5f and 1.0f
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // Tile order: bands of kBandTiles column tiles (4 KB of a row), all row blocks of a band before the next band.  CTAs
    // that run at the same time then add to the sums of many different rows; with whole rows of tiles in flight
    // (112 tiles of a 28672-column matrix adding to the same 32 row sums at once) the row sums cost 20 % of the kernel.
    constexpr int kBandTiles = 8;
    const int tiles_r = (d_out + kPackRows - 1) / kPackRows;
    const int band = blockIdx.x / (kBandTiles * tiles_r);
    const int band_tiles = min(kBandTiles, tiles_c - band * kBandTiles);
    const int in_band = blockIdx.x - band * kBandTiles * tiles_r;
    const int tile_r = in_band / band_tiles, tile_c = band * kBandTiles + (in_band - tile_r * band_tiles);
    const int col0 = tile_c * kTileCols + lane * 8;
    const int row0 = tile_r * kPackRows;
    const int words = d_in >> 5;
    grid_launch_dependents();  // the finalize kernel may be scheduled; it waits for this grid

    uint32_t cunits[8];  // this warp's column sums in units
#pragma unroll
    for (int j = 0; j < 8; ++j) cunits[j] = 0;
    if (row0 + kPackRows <= d_out && (tile_c + 1) * kTileCols <= d_in) {  // CTA-uniform
        uint4 a4[kRowsPerWarp], b4[kRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const size_t idx = (static_cast<size_t>(row0 + warp + 8 * i) * d_in + col0) >> 3;
            a4[i] = ldg_stream(w_f + idx);
            b4[i] = ldg_stream(w_b + idx);
        }
        float cf[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) cf[j] = 0.5f;
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const int o = row0 + warp + 8 * i;
            const uint32_t a[4] = {a4[i].x, a4[i].y, a4[i].z, a4[i].w}, b[4] = {b4[i].x, b4[i].y, b4[i].z, b4[i].w};
            uint32_t spread = 0;
            float rf = 0.5f;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                // bit = (w_f >= w_b): an exact comparison, false for NaN, true for -0 vs +0.  The comparison gives
                // 0xffff per true half; pair p keeps bit 2p of the low half and bit 2p+1 of the high half.
                const uint32_t ge = Elem<BF16>::ge_mask(a[p], b[p]);
                spread |= ge & ((1u << (2 * p)) | (1u << (17 + 2 * p)));
                const float2 fa = Elem<BF16>::to_float2(a[p]), fb = Elem<BF16>::to_float2(b[p]);
                const float d0 = fabsf(__fsub_rz(fa.x, fb.x)), d1 = fabsf(__fsub_rz(fa.y, fb.y));
                if (ROW) rf = __fadd_rz(__fadd_rz(rf, d0), d1);
                if (COL) cf[2 * p] = __fadd_rz(cf[2 * p], d0), cf[2 * p + 1] = __fadd_rz(cf[2 * p + 1], d1);
            }
            uint32_t word = ((spread | (spread >> 16)) & 0xffu) << (8 * (lane & 3));
            word |= __shfl_xor_sync(kFull, word, 1);
            word |= __shfl_xor_sync(kFull, word, 2);
            if ((lane & 3) == 0) mask[static_cast<size_t>(o) * words + (col0 >> 5)] = word;
            if (ROW) {
                const uint32_t rb = __float_as_uint(rf);
                if (__all_sync(kFull, rb < kOneBits)) {  // every lane's sum stayed below 1: exact
                    const uint32_t total = __reduce_add_sync(kFull, rb - kHalfBits);  // <= 32 * 2^23 units
                    if (lane == 0) atomicAdd(row_sum + o, static_cast<unsigned long long>(total));
                } else {
                    pack_row_exact<BF16, true, false>(w_f, w_b, o, col0, d_out, d_in, mask, row_sum, col_sum, lane);
                }
            }
        }
        if (COL) {
            uint32_t worst = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) worst = max(worst, __float_as_uint(cf[j]));
            if (__all_sync(kFull, worst < kOneBits)) {
#pragma unroll
                for (int j = 0; j < 8; ++j) cunits[j] = __float_as_uint(cf[j]) - kHalfBits;
            } else {
                for (int i = 0; i < kRowsPerWarp; ++i)
                    pack_row_exact<BF16, false, true>(w_f, w_b, row0 + warp + 8 * i, col0, d_out, d_in, mask, row_sum, col_sum, lane);
            }
        }
    } else {
        for (int i = 0; i < kRowsPerWarp; ++i)
            pack_row_exact<BF16, ROW, COL>(w_f, w_b, row0 + warp + 8 * i, col0, d_out, d_in, mask, row_sum, col_sum, lane);
    }
    if (COL) {
#pragma unroll
        for (int j = 0; j < 8; ++j) s_col[warp * kTileCols + lane * 8 + j] = cunits[j];
        __syncthreads();
        const int c = tile_c * kTileCols + threadIdx.x;
        if (c < d_in) {
            uint32_t sum = 0;  // <= 32 rows * 2^23 units
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) sum += s_col[w * kTileCols + threadIdx.x];
            if (sum) atomicAdd(col_sum + c, static_cast<unsigned long long>(sum));
        }
    }
}

// Sums -> scales, and the sums go back to zero: the scratch area is left as it was found.
__global__ void pack_finalize_kernel(unsigned long long *__restrict__ row_sum, unsigned long long *__restrict__ col_sum,
                                     int d_out, int d_in, unsigned short *__restrict__ v_row,
                                     unsigned short *__restrict__ v_col) {
    grid_dependency_wait();  // every tile has added its sums
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const bool is_row = idx < d_out;
    const int j = is_row ? idx : idx - d_out;
    if (!is_row && j >= d_in) return;
    unsigned long long *src = (is_row ? row_sum : col_sum) + j;
    unsigned short *dst = is_row ? v_row : v_col;
    if (dst == nullptr) return;  // that axis was not asked for: its sums were never touched
    const unsigned long long sum = *src;
    *src = 0ull;
    dst[j] = mean_to_half(sum, is_row ? d_in : d_out);
}

template <bool BF16, int AXIS>
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
            const float2 f = Elem<false>::to_float2(u[p]);  // the scales are binary16
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
            const float2 f = Elem<BF16>::to_float2(w[p]);
            const float s0 = __uint_as_float(__float_as_uint(vf[2 * p]) ^ (((nbits >> (2 * p)) & 1u) << 31));
            const float s1 = __uint_as_float(__float_as_uint(vf[2 * p + 1]) ^ (((nbits >> (2 * p + 1)) & 1u) << 31));
            r[p] = Elem<BF16>::from_float2(__fadd_rn(f.x, s0), __fadd_rn(f.y, s1));  // one fp32 add, one rounding to 16 bits
        }
        stg_stream(w_hat + idx, make_uint4(r[0], r[1], r[2], r[3]));
    }
}

}  // namespace

size_t pack_scratch_bytes(int64_t d_out, int64_t d_in) {
    return round_up(sizeof(unsigned long long) * static_cast<size_t>(d_out + d_in), 256);
}

// scratch: pack_scratch_bytes() bytes, all zero on entry; the call leaves them zero again.
pd_status launch_pack(const __half *w_f, const __half *w_b, int64_t d_out, int64_t d_in, uint32_t *mask,
                      __half *v_row, __half *v_col, unsigned long long *sums, bool bf16, cudaStream_t stream) {
    unsigned long long *row_sum = sums, *col_sum = sums + d_out;
    const int tiles_c = static_cast<int>((d_in + kTileCols - 1) / kTileCols);
    const int64_t tiles = ((d_out + kPackRows - 1) / kPackRows) * tiles_c;
    if (tiles > INT_MAX / 2) return PD_ERR_UNSUPPORTED_SHAPE;
    const unsigned grid = static_cast<unsigned>(tiles);
    const uint4 *a = reinterpret_cast<const uint4 *>(w_f), *b = reinterpret_cast<const uint4 *>(w_b);
    const int n_out = static_cast<int>(d_out), n_in = static_cast<int>(d_in);
#define PD_PACK(BF, R, C) pack_kernel<BF, R, C><<<grid, kThreads, 0, stream>>>(a, b, n_out, n_in, tiles_c, mask, row_sum, col_sum)
    if (bf16) {
        if (v_row && v_col) PD_PACK(true, true, true);
        else if (v_row) PD_PACK(true, true, false);
        else PD_PACK(true, false, true);
    } else {
        if (v_row && v_col) PD_PACK(false, true, true);
        else if (v_row) PD_PACK(false, true, false);
        else PD_PACK(false, false, true);
    }
#undef PD_PACK
    if (cudaGetLastError() != cudaSuccess) return PD_ERR_CUDA;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may be scheduled while the pack kernel runs
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>((d_out + d_in + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch(2);
    return cuda_ok(cudaLaunchKernelEx(&cfg, pack_finalize_kernel, row_sum, col_sum, n_out, n_in,
                                      reinterpret_cast<unsigned short *>(v_row), reinterpret_cast<unsigned short *>(v_col)));
}

pd_status launch_merge(const __half *w_b, const uint32_t *mask, const __half *v, int axis, int64_t d_out,
                       int64_t d_in, __half *w_hat, bool bf16, cudaStream_t stream) {
    const int tiles_c = static_cast<int>((d_in + kTileCols - 1) / kTileCols);
    const int64_t tiles = ((d_out + kTileRows - 1) / kTileRows) * tiles_c;
    const dim3 grid(static_cast<unsigned>(tiles)), block(kThreads);
    const uint4 *b = reinterpret_cast<const uint4 *>(w_b);
    uint4 *out = reinterpret_cast<uint4 *>(w_hat);
#define PD_MERGE(BF, AX) merge_kernel<BF, AX><<<grid, block, 0, stream>>>(b, mask, v, (int)d_out, (int)d_in, tiles_c, out)
    if (bf16) {
        if (axis == PD_AXIS_ROW) PD_MERGE(true, PD_AXIS_ROW);
        else PD_MERGE(true, PD_AXIS_COL);
    } else {
        if (axis == PD_AXIS_ROW) PD_MERGE(false, PD_AXIS_ROW);
        else PD_MERGE(false, PD_AXIS_COL);
    }
#undef PD_MERGE
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
    // the array starts zero-filled (device globals do) and every call puts what it used back to zero
    return launch_pack(static_cast<const __half *>(w_f), static_cast<const __half *>(w_b), d_out, d_in, mask,
                       static_cast<__half *>(v_row), static_cast<__half *>(v_col), sums, false,
                       static_cast<cudaStream_t>(cuda_stream));
}
