// Fitting the scale vector of one layer by output matching (paper, section "Calibration cache, training, and
// stacking": L = (1/n) ||Y - Y_hat||^2 minimised over v with AdamW; Algorithm "Train per-row/column scaling vectors
// via activation matching").  W_b and the sign mask B stay fixed, so one training step is
//
//   row axis :  Z = X W_b^T,  P = X B^T,  R = Z + v[o] P - Y,          dL/dv[o] = (2/n) sum_m R[m,o] P[m,o]
//   col axis :  R = X W_b^T + X (v (.) B)^T - Y,   T = R B,            dL/dv[i] = (2/n) sum_m X[m,i] T[m,i]
//   scalar   :  the row formulas with one v for the whole matrix,      dL/dv    = sum of the row gradients
//
// Every product runs on the 5th-generation tensor cores with fp32 accumulation; W_b and B are separate operands
// (B as exact +-1, or +-binary16(v[i]) for the col axis), so the delta term is not rounded into the weights.
// One kernel, three modes:
//   FIT_ROW_FWD : two accumulators (Z, P) per tile of 128 rows x 192 tokens; the epilogue forms R, the squared
//                 error and the row gradient without writing R anywhere
//   FIT_COL_FWD : one accumulator; the epilogue writes R as binary16 for the second pass
//   FIT_COL_BWD : T^T = B^T R^T from the transposed mask (rows = input columns); the epilogue multiplies by X
// About half of a k step's time does not depend on the number of tokens, so the tiles are as wide in tokens as tensor
// memory allows in the row mode: 2 x 192 accumulator columns + the sign ring (4 x 32).  The tile of Y (of X in the
// backward mode) that the epilogue needs is fetched into shared memory with cp.async while the tile's MMAs run:
// read element by element from global memory it cost 40 % of the kernel's time.
// The W_b tile is an MMA operand straight from the shared memory TMA filled (A from a shared-memory descriptor);
// only the sign rows go through tensor memory: a thread of the eight transform warps owns one row (= one TMEM lane)
// and expands two mask words per 64-wide k step.  Roles: warp 0 TMA (token tile, W_b tile, the col-axis scales of
// the step), warp 1 MMA issue, warps 2-5 epilogue, warps 6-13 transform.  Four k steps are in flight.  Partial sums
// go to the workspace per tile and are added in a fixed order by fit_reduce_kernel: results do not depend on the
// schedule.  Every wait is bounded.
#include "pd_tcgen05.cuh"

namespace pd {
namespace {

constexpr int FM = 128;           // rows of the weight-side operand per tile (MMA M, TMEM lanes)
constexpr int FK = 64;            // k per step
constexpr int kFitStages = 4;     // token ring, W_b ring and sign ring (tensor memory)
constexpr int kFitWarps = 14;
constexpr int kFitThreads = kFitWarps * 32;
constexpr int kFitXformWarps = 8;
constexpr int kFitEpiWarps = 4;
constexpr int kFitACol0 = 384;        // sign ring: kFitStages slots of 32 TMEM columns
constexpr uint32_t kOnesF16 = 0x3C003C00u;

enum FitMode { FIT_ROW_FWD = 0, FIT_COL_FWD = 1, FIT_COL_BWD = 2 };
// tokens per tile (MMA N): the row mode keeps two accumulators in 384 of the 512 tensor-memory columns
__host__ __device__ constexpr int fit_tokens(int) { return 192; }

struct FitArgs {
    const uint32_t *bits;  // forward: mask [d_out][d_in/32]; backward: transposed mask [d_in][words_t]
    int words;             // words per row of `bits`
    const float *v;        // row forward: scales [d_out], or one entry when `scalar`
    const __half *v16;     // col forward: binary16 copy of the scales [d_in]
    const __half *y;       // forward: targets [M][d_out]
    const __half *x;       // backward: inputs [M][d_in]
    __half *resid;         // col forward writes the residual [M][ld_r]; the backward pass reads it through its tensor map
    int ld_r;
    float *part_g;         // [token tiles][rows] partial gradient sums (before the factor 2/n)
    float *part_loss;      // forward: [tiles] partial sums of squared residuals
    int M, rows, K;        // rows of the weight-side operand (d_out forward, d_in backward); contraction length
    int tiles_m, tiles_n, k_steps;
    int scalar;
    uint32_t *status;
};

struct FitSmem {
    static constexpr int kXBytes = fit_tokens(0) * FK * 2;   // 24 KB
    static constexpr int kWBytes = FM * FK * 2;              // 16 KB
    static constexpr int kXOffset = 0;
    static constexpr int kWOffset = kFitStages * kXBytes;
    static constexpr int kYOffset = kWOffset + kFitStages * kWBytes;   // [token][128 rows] binary16: the epilogue's Y (or X) tile
    static constexpr int kYBytes = fit_tokens(0) * FM * 2;   // 48 KB
    static constexpr int kBarOffset = kYOffset + kYBytes;
    static constexpr int kVOffset = kBarOffset + 256;          // col forward: the 64 scales of a k step, per stage
    static constexpr int kRedOffset = kVOffset + kFitStages * 128;
    static constexpr int kTotal = kRedOffset + 64 + 1024;      // + slack for 1024-byte alignment
    static_assert(kTotal <= 227 * 1024, "shared memory per CTA");
};

// A from shared memory (K-major tile, 128-byte swizzle, like B)
__device__ __forceinline__ void tcgen05_mma_f16_smem_a(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 64 signs (two mask words) -> 32 registers of two binary16 each: +mag where the bit is 1, -mag where it is 0.
// COL: mag = the step's 64 scales from shared memory; else mag = 1.
template <bool COL>
__device__ __forceinline__ void build_sign_row(uint32_t (&out)[32], const unsigned char *vs, uint32_t word0, uint32_t word1) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t vv[4] = {kOnesF16, kOnesF16, kOnesF16, kOnesF16};
        if (COL) {
            const uint4 t4 = *reinterpret_cast<const uint4 *>(vs + 16 * c);
            vv[0] = t4.x, vv[1] = t4.y, vv[2] = t4.z, vv[3] = t4.w;
        }
        // byte c & 3 of the word holds the 8 signs of this piece; b * 0x8001 puts bit i at i and i + 15
        const uint32_t sp = prmt(c < 4 ? word0 : word1, 0u, 0x4440u | static_cast<uint32_t>(c & 3)) * 0x8001u;
#pragma unroll
        for (int pr = 0; pr < 4; ++pr) out[4 * c + pr] = lop3_andn_xor(sp << (15 - 2 * pr), 0x80008000u, vv[pr]);
    }
}

template <int MODE>
__global__ void __launch_bounds__(kFitThreads, 1)
fit_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const FitArgs a) {
    constexpr bool FWD = MODE != FIT_COL_BWD;
    constexpr int BN = fit_tokens(MODE);
    constexpr uint32_t kAccP = BN;  // TMEM column of the second accumulator (row mode)
    static_assert((MODE == FIT_ROW_FWD ? 2 : 1) * BN <= kFitACol0, "accumulators end where the sign ring starts");
    using L = FitSmem;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBarOffset);
    uint64_t *v_full = bars;                       // col forward: the step's scales have landed
    uint64_t *ready = bars + kFitStages;           // token tile and W_b tile landed (TMA bytes + the producer's arrival), sign slot written
    uint64_t *consumed = bars + 2 * kFitStages;    // the MMAs of the step have read its shared-memory tiles and its sign slot
    uint64_t *acc_full = bars + 3 * kFitStages, *acc_empty = acc_full + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    float *red = reinterpret_cast<float *>(smem + L::kRedOffset);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = a.tiles_m * a.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFitStages; ++s) {
            mbar_init(v_full + s, 1);
            mbar_init(ready + s, kFitXformWarps / 2 + 1);
            mbar_init(consumed + s, 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, kFitEpiWarps);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (threadIdx.x < kFitStages * 128 / 4) {  // a short last k step leaves the tail of its scale slot untouched
        reinterpret_cast<uint32_t *>(smem + L::kVOffset)[threadIdx.x] = 0u;
        fence_proxy_async_smem();
    }
    if (warp == 1) tcgen05_alloc(tmem_slot, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer: token tile, W_b tile, col-axis scales of the step
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const int tm = tile / a.tiles_n, tn = tile - tm * a.tiles_n;
                for (int ks = 0; ks < a.k_steps; ++ks, ++it) {
                    const int s = it % kFitStages;
                    const uint32_t round = it / kFitStages;
                    // the slots were last read by k step it - kFitStages
                    if (round > 0 && !(ok = mbar_wait(consumed + s, (round - 1) & 1, abort_flag, a.status, 31))) break;
                    if (MODE == FIT_COL_FWD) {
                        const uint32_t v_bytes = static_cast<uint32_t>(min(FK, a.K - ks * FK) * 2);
                        mbar_arrive_expect_tx(v_full + s, v_bytes);
                        bulk_load_1d(smem + L::kVOffset + s * 128, a.v16 + static_cast<size_t>(ks) * FK, v_bytes, v_full + s);
                    }
                    mbar_arrive_expect_tx(ready + s, BN * FK * 2 + (FWD ? L::kWBytes : 0));
                    tma_load_2d(&map_x, ready + s, smem + L::kXOffset + s * L::kXBytes, ks * FK, tn * BN);
                    if (FWD) tma_load_2d(&map_w, ready + s, smem + L::kWOffset + s * L::kWBytes, ks * FK, tm * FM);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = kIdescBase<false> | (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(FM >> 4) << 24);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tcount) {
                if (!(ok = mbar_wait(acc_empty, (tcount & 1) ^ 1, abort_flag, a.status, 33))) break;
                tcgen05_fence_after();
                for (int ks = 0; ks < a.k_steps; ++ks, ++it) {
                    const int s = it % kFitStages;
                    if (!(ok = mbar_wait(ready + s, (it / kFitStages) & 1, abort_flag, a.status, 34))) break;
                    tcgen05_fence_after();
                    const uint32_t x_addr = smem_u32(smem + L::kXOffset + s * L::kXBytes);
                    const uint32_t w_addr = smem_u32(smem + L::kWOffset + s * L::kWBytes);
                    const uint32_t a_s = tmem_base + kFitACol0 + s * 32;
#pragma unroll
                    for (int kk = 0; kk < FK / 16; ++kk) {
                        const uint64_t xd = make_smem_desc(x_addr + kk * 32);
                        const uint32_t first = (ks > 0 || kk > 0) ? 1u : 0u;
                        if (MODE == FIT_ROW_FWD) {
                            tcgen05_mma_f16_smem_a(tmem_base, make_smem_desc(w_addr + kk * 32), xd, idesc, first);
                            tcgen05_mma_f16_tmem_a(tmem_base + kAccP, a_s + kk * 8, xd, idesc, first);
                        } else if (MODE == FIT_COL_FWD) {
                            tcgen05_mma_f16_smem_a(tmem_base, make_smem_desc(w_addr + kk * 32), xd, idesc, first);
                            tcgen05_mma_f16_tmem_a(tmem_base, a_s + kk * 8, xd, idesc, 1u);
                        } else {
                            tcgen05_mma_f16_tmem_a(tmem_base, a_s + kk * 8, xd, idesc, first);
                        }
                    }
                    tcgen05_commit(consumed + s);
                }
                if (ok) tcgen05_commit(acc_full);
            }
        }
    } else if (warp < 2 + kFitEpiWarps) {
        // ------------------------------------------------ epilogue: a thread owns one row of the tile and walks its tokens
        const int quarter = warp & 3;
        const int et = threadIdx.x - 2 * 32;  // 0..127 among the epilogue threads
        const unsigned char *ybuf = smem + L::kYOffset;
        const __half *side = FWD ? a.y : a.x;  // [M][rows]: the operand the epilogue combines with the accumulator
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tcount) {
            const int tm = tile / a.tiles_n, tn = tile - tm * a.tiles_n;
            {   // this tile's [tokens][128 rows] piece of `side`, 16 bytes per copy, while the MMAs run
                const int n_tok = min(BN, a.M - tn * BN);
                for (int idx = et; idx < n_tok * 16; idx += kFitEpiWarps * 32) {
                    const int tok = idx >> 4, ch = idx & 15;
                    const int r8 = tm * FM + ch * 8;
                    if (r8 < a.rows)  // rows is a multiple of 8: a piece is valid as a whole or not at all
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(ybuf + tok * (FM * 2) + ch * 16)),
                                     "l"(side + static_cast<size_t>(tn * BN + tok) * a.rows + r8)
                                     : "memory");
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            }
            const bool got = mbar_wait(acc_full, tcount & 1, abort_flag, a.status, 35);
            uint32_t gave_up;  // OR over the epilogue warps, so that they leave together
            asm volatile(
                "{\n"
                ".reg .pred p, q;\n"
                "setp.ne.u32 q, %1, 0;\n"
                "bar.red.or.pred p, 2, %2, q;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(gave_up)
                : "r"(static_cast<uint32_t>(!got)), "n"(kFitEpiWarps * 32)
                : "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            if (gave_up) break;
            asm volatile("bar.sync 2, %0;" ::"n"(kFitEpiWarps * 32) : "memory");  // every thread's copies have landed
            tcgen05_fence_after();
            const int row = tm * FM + quarter * 32 + lane;
            const bool row_ok = row < a.rows;
            const __half *ycol = reinterpret_cast<const __half *>(ybuf) + quarter * 32 + lane;  // + token * FM
            const int tok0 = tn * BN;
            const int count = min(BN, a.M - tok0);
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            float vo = 0.f;
            if (MODE == FIT_ROW_FWD && row_ok) vo = __ldg(a.v + (a.scalar ? 0 : row));
            float g_acc = 0.f, l_acc = 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (c0 >= count) break;  // warp-uniform
                uint32_t z[32];
                tcgen05_ld_32x32b_x32(taddr + c0, z);
                if (MODE == FIT_ROW_FWD) {
                    uint32_t p[32];
                    tcgen05_ld_32x32b_x32(taddr + kAccP + c0, p);
                    tcgen05_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int tok = tok0 + c0 + j;
                        if (row_ok && tok < a.M) {
                            const float yv = __half2float(ycol[(c0 + j) * FM]);
                            const float pj = __uint_as_float(p[j]);
                            const float r = fmaf(vo, pj, __uint_as_float(z[j])) - yv;
                            l_acc = fmaf(r, r, l_acc);
                            g_acc = fmaf(r, pj, g_acc);
                        }
                    }
                } else if (MODE == FIT_COL_FWD) {
                    tcgen05_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int tok = tok0 + c0 + j;
                        if (row_ok && tok < a.M) {
                            const float yv = __half2float(ycol[(c0 + j) * FM]);
                            const float r = __uint_as_float(z[j]) - yv;
                            l_acc = fmaf(r, r, l_acc);
                            // the residual takes y's place in the shared-memory tile (this thread alone touches the entry)
                            const_cast<__half *>(ycol)[(c0 + j) * FM] = __float2half_rn(r);
                        }
                    }
                } else {
                    tcgen05_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int tok = tok0 + c0 + j;
                        if (row_ok && tok < a.M) {
                            const float xv = __half2float(ycol[(c0 + j) * FM]);
                            g_acc = fmaf(xv, __uint_as_float(z[j]), g_acc);
                        }
                    }
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);
            if (MODE == FIT_COL_FWD) {  // the residual tile leaves with 16-byte stores, 256 contiguous bytes per token
                asm volatile("bar.sync 2, %0;" ::"n"(kFitEpiWarps * 32) : "memory");
                for (int idx = et; idx < count * 16; idx += kFitEpiWarps * 32) {
                    const int tok = idx >> 4, ch = idx & 15;
                    const int r8 = tm * FM + ch * 8;
                    if (r8 < a.rows)
                        *reinterpret_cast<uint4 *>(a.resid + static_cast<size_t>(tok0 + tok) * a.ld_r + r8) =
                            *reinterpret_cast<const uint4 *>(ybuf + tok * (FM * 2) + ch * 16);
                }
            }
            if (MODE != FIT_COL_FWD && row_ok) a.part_g[static_cast<size_t>(tn) * a.rows + row] = g_acc;
            if (!FWD) asm volatile("bar.sync 2, %0;" ::"n"(kFitEpiWarps * 32) : "memory");  // the tile in shared memory is free again
            if (FWD) {  // squared error of the tile: lanes in a fixed tree, then the four warps in order
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) l_acc += __shfl_xor_sync(0xffffffffu, l_acc, d);
                if (lane == 0) red[quarter] = l_acc;
                asm volatile("bar.sync 2, %0;" ::"n"(kFitEpiWarps * 32) : "memory");
                if (quarter == 0 && lane == 0) a.part_loss[tile] = (red[0] + red[1]) + (red[2] + red[3]);
                asm volatile("bar.sync 2, %0;" ::"n"(kFitEpiWarps * 32) : "memory");
            }
        }
    } else {
        // ------------------------------------------------ transform: the sign rows of a k step -> its slot in tensor memory
        const int quarter = warp & 3;
        const uint32_t par = static_cast<uint32_t>((warp - (2 + kFitEpiWarps)) >> 2);  // four warps take the even steps, four the odd ones
        const int r = quarter * 32 + lane;
        const uint32_t a_taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + kFitACol0;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            const int tm = tile / a.tiles_n;
            const int row = tm * FM + r;
            const bool row_ok = row < a.rows;
            const uint32_t *mrow = a.bits + static_cast<size_t>(row_ok ? row : 0) * a.words;
            auto load_words = [&](int ks, uint32_t &w0, uint32_t &w1) {
                w0 = (row_ok && ks < a.k_steps && 2 * ks < a.words) ? __ldg(mrow + 2 * ks) : 0u;
                w1 = (row_ok && ks < a.k_steps && 2 * ks + 1 < a.words) ? __ldg(mrow + 2 * ks + 1) : 0u;
            };
            int ks = static_cast<int>((par ^ it) & 1u);  // first k step of this tile that falls to this warp
            uint32_t q0[4], q1[4];
#pragma unroll
            for (int d = 0; d < 4; ++d) load_words(ks + 2 * d, q0[d], q1[d]);
            for (; ks < a.k_steps; ks += 2) {
                const uint32_t my_it = it + ks;
                const int s = my_it % kFitStages;
                const uint32_t round = my_it / kFitStages;
                const uint32_t word0 = q0[0], word1 = q1[0];
#pragma unroll
                for (int d = 0; d < 3; ++d) q0[d] = q0[d + 1], q1[d] = q1[d + 1];
                load_words(ks + 8, q0[3], q1[3]);
                uint32_t out[32];
                if (MODE == FIT_COL_FWD) {
                    if (!(ok = __all_sync(0xffffffffu, mbar_wait(v_full + s, round & 1, abort_flag, a.status, 36)))) break;
                    build_sign_row<true>(out, smem + L::kVOffset + s * 128, word0, word1);
                } else {
                    build_sign_row<false>(out, nullptr, word0, word1);
                }
                // the slot was last read by the MMAs of k step my_it - kFitStages
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(consumed + s, (round & 1) ^ 1, abort_flag, a.status, 37)))) break;
                tcgen05_fence_after();
                tcgen05_st_32x32b_x32(a_taddr + s * 32, out);
                tcgen05_wait_st();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(ready + s);
            }
            it += a.k_steps;
        }
    }

    // ------------------------------------------------ teardown
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);  // copies that may still be in flight
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, 512);
    }
}

// Adds the per-tile partial sums in a fixed order (double accumulation) and applies the factors of the mean:
// grad[k] = (2/n) sum over token tiles of part_g[tile][k]; the block after the gradient blocks writes
// loss = (1/n) sum of part_loss and, in scalar mode, the single gradient entry = sum over all rows.
__global__ void __launch_bounds__(256)
fit_reduce_kernel(const float *part_g, int tiles_tok, int rows, float *grad, int scalar, const float *part_loss, int n_loss,
                  float *loss, double inv_n, int g_blocks) {
    __shared__ double red[256];
    if (static_cast<int>(blockIdx.x) < g_blocks) {
        const int k = blockIdx.x * 256 + threadIdx.x;
        if (k < rows) {
            double acc = 0.0;
            for (int t = 0; t < tiles_tok; ++t) acc += static_cast<double>(part_g[static_cast<size_t>(t) * rows + k]);
            grad[k] = static_cast<float>(2.0 * inv_n * acc);
        }
        return;
    }
    for (int pass = 0; pass < 2; ++pass) {
        if (pass == 0 && loss == nullptr) continue;
        if (pass == 1 && !(scalar && grad != nullptr)) continue;
        double acc = 0.0;
        if (pass == 0) {
            for (int i = threadIdx.x; i < n_loss; i += 256) acc += static_cast<double>(part_loss[i]);
        } else {
            for (int k = threadIdx.x; k < rows; k += 256)
                for (int t = 0; t < tiles_tok; ++t) acc += static_cast<double>(part_g[static_cast<size_t>(t) * rows + k]);
        }
        red[threadIdx.x] = acc;
        __syncthreads();
        for (int d = 128; d > 0; d >>= 1) {
            if (static_cast<int>(threadIdx.x) < d) red[threadIdx.x] += red[threadIdx.x + d];
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            if (pass == 0) *loss = static_cast<float>(inv_n * red[0]);
            else grad[0] = static_cast<float>(2.0 * inv_n * red[0]);
        }
        __syncthreads();
    }
}

// One AdamW step (decoupled weight decay, bias-corrected moments) on fp32 state; also refreshes the binary16 copy of
// the scales that the col-axis forward pass multiplies with.  lr == 0 and t == 0: only the copy is written.
__global__ void __launch_bounds__(256)
fit_adamw_kernel(float *v, float *m1, float *m2, const float *g, int len, float lr, float b1, float b2, float eps, float wd,
                 float inv_c1, float inv_c2, __half *v16, int update) {
    const int k = blockIdx.x * 256 + threadIdx.x;
    if (k >= len) return;
    float vk = v[k];
    if (update) {
        const float gk = g[k];
        vk *= 1.0f - lr * wd;
        const float m = b1 * m1[k] + (1.0f - b1) * gk;
        const float s = b2 * m2[k] + (1.0f - b2) * gk * gk;
        m1[k] = m, m2[k] = s;
        vk -= lr * (m * inv_c1) / (sqrtf(s * inv_c2) + eps);
        v[k] = vk;
    }
    if (v16) v16[k] = __float2half_rn(vk);
}

// binary16 -> fp32 state: v from the packed artifact's scales, zero moments
__global__ void __launch_bounds__(256) fit_init_kernel(const __half *v16, float *v, float *m1, float *m2, int len) {
    const int k = blockIdx.x * 256 + threadIdx.x;
    if (k >= len) return;
    v[k] = __half2float(v16[k]);
    m1[k] = 0.f, m2[k] = 0.f;
}

// Transposed bit mask: out[i][o / 32] bit (o % 32) = mask[o][i / 32] bit (i % 32).  A warp transposes one 32 x 32 block
// with 32 ballots; rows past d_out read as zero bits.
__global__ void __launch_bounds__(128)
transpose_mask_kernel(const uint32_t *mask, int d_out, int words_in, uint32_t *out, int words_out) {
    const int lane = threadIdx.x & 31;
    const int w = blockIdx.x * 4 + (threadIdx.x >> 5);  // word column of the input
    const int ob = blockIdx.y;                           // block of 32 input rows = word column of the output
    if (w >= words_in) return;                           // warp-uniform
    const int o = ob * 32 + lane;
    const uint32_t word = o < d_out ? __ldg(mask + static_cast<size_t>(o) * words_in + w) : 0u;
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const uint32_t b = __ballot_sync(0xffffffffu, (word >> j) & 1u);
        if (lane == j) mine = b;
    }
    out[static_cast<size_t>(w * 32 + lane) * words_out + ob] = mine;
}

// Row/Col selection (Algorithm "Per-layer compression with Row/Col selection": row when E_row <= E_col) and the
// chosen scales as binary16.
__global__ void __launch_bounds__(256)
fit_select_kernel(const float *val_loss, const float *v_row, int d_out, const float *v_col, int d_in, __half *v_out, int32_t *axis_out) {
    const bool row = val_loss[0] <= val_loss[1];
    const int len = row ? d_out : d_in;
    const float *src = row ? v_row : v_col;
    for (int k = blockIdx.x * 256 + threadIdx.x; k < len; k += gridDim.x * 256) v_out[k] = __float2half_rn(src[k]);
    if (blockIdx.x == 0 && threadIdx.x == 0) *axis_out = row ? PD_AXIS_ROW : PD_AXIS_COL;
}

bool make_fit_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    return make_map_2d(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, rows, cols, ld * 2, FK, box_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

template <int MODE>
pd_status launch_fit_gemm(const CUtensorMap &mw, const CUtensorMap &mx, const FitArgs &args, cudaStream_t stream) {
    auto kernel = fit_gemm_kernel<MODE>;
    static std::atomic<bool> configured[kMaxDevices];
    if (!ensure_dynamic_smem(kernel, FitSmem::kTotal, configured)) return PD_ERR_CUDA;
    const int tiles = args.tiles_m * args.tiles_n;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    kernel<<<grid, kFitThreads, FitSmem::kTotal, stream>>>(mw, mx, args);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

struct FitScratch {
    float *part_loss, *part_g;
    __half *resid, *v16;
    size_t total;
};

FitScratch carve_fit_scratch(unsigned char *base, int64_t M, int64_t d_out, int64_t d_in) {
    const int64_t tiles_tok = (M + fit_tokens(FIT_ROW_FWD) - 1) / fit_tokens(FIT_ROW_FWD), tiles_o = (d_out + FM - 1) / FM;  // the narrowest token tile
    const int64_t maxdim = d_out > d_in ? d_out : d_in;
    FitScratch s;
    size_t off = 0;
    s.part_loss = reinterpret_cast<float *>(base + off);
    off += round_up(static_cast<size_t>(tiles_tok * tiles_o) * 4, 256);
    s.part_g = reinterpret_cast<float *>(base + off);
    off += round_up(static_cast<size_t>(tiles_tok * maxdim) * 4, 256);
    s.resid = reinterpret_cast<__half *>(base + off);
    off += round_up(static_cast<size_t>(M) * round_up(static_cast<size_t>(d_out), 8) * 2, 256);
    s.v16 = reinterpret_cast<__half *>(base + off);
    off += round_up(static_cast<size_t>(d_in) * 2, 256);
    s.total = off;
    return s;
}

}  // namespace

size_t fit_scratch_bytes(int64_t M, int64_t d_out, int64_t d_in) { return carve_fit_scratch(nullptr, M, d_out, d_in).total; }

pd_status launch_transpose_mask(const uint32_t *mask, int64_t d_out, int64_t d_in, uint32_t *mask_t, cudaStream_t stream) {
    const int words_in = static_cast<int>(d_in / 32), words_out = static_cast<int>((d_out + 31) / 32);
    dim3 grid(static_cast<unsigned>((words_in + 3) / 4), static_cast<unsigned>(words_out));
    transpose_mask_kernel<<<grid, 128, 0, stream>>>(mask, static_cast<int>(d_out), words_in, mask_t, words_out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

pd_status launch_fit_adamw(float *v, float *m1, float *m2, const float *g, int64_t len, int64_t t, float lr, float b1, float b2,
                           float eps, float wd, __half *v16, cudaStream_t stream) {
    const double c1 = 1.0 - pow(static_cast<double>(b1), static_cast<double>(t));
    const double c2 = 1.0 - pow(static_cast<double>(b2), static_cast<double>(t));
    const int update = t > 0 ? 1 : 0;
    fit_adamw_kernel<<<static_cast<unsigned>((len + 255) / 256), 256, 0, stream>>>(
        v, m1, m2, g, static_cast<int>(len), lr, b1, b2, eps, wd, update ? static_cast<float>(1.0 / c1) : 0.f,
        update ? static_cast<float>(1.0 / c2) : 0.f, v16, update);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

// loss (and, with grad != nullptr, its gradient) of one batch.  axis: PD_AXIS_ROW, PD_AXIS_COL or PD_AXIS_SCALAR.
pd_status launch_fit_loss_grad(const __half *x, const __half *y, int64_t M, const __half *w_b, const uint32_t *mask,
                               const uint32_t *mask_t, const float *v, int axis, int64_t d_out, int64_t d_in, float *loss,
                               float *grad, unsigned char *scratch, uint32_t *status, cudaStream_t stream) {
    const FitScratch sc = carve_fit_scratch(scratch, M, d_out, d_in);
    const int bn = fit_tokens(axis == PD_AXIS_COL ? FIT_COL_FWD : FIT_ROW_FWD);
    const int tiles_tok = static_cast<int>((M + bn - 1) / bn);
    const int64_t ld_r = static_cast<int64_t>(round_up(static_cast<size_t>(d_out), 8));
    const double inv_n = 1.0 / (static_cast<double>(M) * static_cast<double>(d_out));
    CUtensorMap mw, mx;
    if (!make_fit_map(&mw, w_b, d_out, d_in, d_in, FM) || !make_fit_map(&mx, x, M, d_in, d_in, bn)) return PD_ERR_CUDA;
    FitArgs a = {};
    a.bits = mask;
    a.words = static_cast<int>(d_in / 32);
    a.v = v;
    a.v16 = sc.v16;
    a.y = y;
    a.x = x;
    a.resid = sc.resid;
    a.ld_r = static_cast<int>(ld_r);
    a.part_g = sc.part_g;
    a.part_loss = sc.part_loss;
    a.M = static_cast<int>(M);
    a.rows = static_cast<int>(d_out);
    a.K = static_cast<int>(d_in);
    a.tiles_m = static_cast<int>((d_out + FM - 1) / FM);
    a.tiles_n = tiles_tok;
    a.k_steps = static_cast<int>((d_in + FK - 1) / FK);
    a.scalar = axis == PD_AXIS_SCALAR ? 1 : 0;
    a.status = status;
    const int n_loss = a.tiles_m * a.tiles_n;
    pd_status st;
    if (axis != PD_AXIS_COL) {
        if ((st = launch_fit_gemm<FIT_ROW_FWD>(mw, mx, a, stream)) != PD_OK) return st;
        const int g_blocks = (grad && !a.scalar) ? static_cast<int>((d_out + 255) / 256) : 0;
        fit_reduce_kernel<<<g_blocks + 1, 256, 0, stream>>>(sc.part_g, tiles_tok, static_cast<int>(d_out), grad, a.scalar,
                                                            sc.part_loss, n_loss, loss, inv_n, g_blocks);
        count_launch();
        return cuda_ok(cudaGetLastError());
    }
    // col axis: binary16 copy of the scales, forward pass with the residual written out, then R B through the transposed mask
    if ((st = launch_fit_adamw(const_cast<float *>(v), nullptr, nullptr, nullptr, d_in, 0, 0.f, 0.f, 0.f, 0.f, 0.f, sc.v16, stream)) != PD_OK)
        return st;
    if ((st = launch_fit_gemm<FIT_COL_FWD>(mw, mx, a, stream)) != PD_OK) return st;
    int g_blocks = 0;
    if (grad) {
        CUtensorMap mr;
        if (!make_fit_map(&mr, sc.resid, M, d_out, ld_r, fit_tokens(FIT_COL_BWD))) return PD_ERR_CUDA;
        FitArgs b = a;
        b.bits = mask_t;
        b.words = static_cast<int>((d_out + 31) / 32);
        b.rows = static_cast<int>(d_in);
        b.K = static_cast<int>(d_out);
        b.tiles_m = static_cast<int>((d_in + FM - 1) / FM);
        b.k_steps = static_cast<int>((d_out + FK - 1) / FK);
        if ((st = launch_fit_gemm<FIT_COL_BWD>(mr, mr, b, stream)) != PD_OK) return st;
        g_blocks = static_cast<int>((d_in + 255) / 256);
    }
    fit_reduce_kernel<<<g_blocks + 1, 256, 0, stream>>>(sc.part_g, tiles_tok, static_cast<int>(d_in), grad, 0, sc.part_loss, n_loss,
                                                        loss, inv_n, g_blocks);
    count_launch();
    return cuda_ok(cudaGetLastError());
}


size_t fit_layer_scratch_bytes(int64_t m_batch, int64_t m_val, int64_t d_out, int64_t d_in) {
    const int64_t m = m_batch > m_val ? m_batch : m_val;
    return fit_scratch_bytes(m, d_out, d_in) + round_up(static_cast<size_t>(d_in) * ((d_out + 31) / 32) * 4, 256) +
           round_up(static_cast<size_t>(4 * (d_out + d_in)) * 4, 256) + 256;
}

// Algorithm "Per-layer compression with Row/Col selection": both axis variants start from the packed artifact's
// scales, are trained with the same budget (Algorithm "Train per-row/column scaling vectors": epochs x minibatches,
// AdamW on v only, optional cosine schedule over all steps), and the one with the lower validation loss is kept
// (row on a tie).  Everything is enqueued on `stream`; nothing synchronises.
pd_status launch_fit_layer(const __half *x_tr, const __half *y_tr, int64_t m_tr, const __half *x_val, const __half *y_val,
                           int64_t m_val, const __half *w_b, const uint32_t *mask, const __half *v_row0, const __half *v_col0,
                           int64_t d_out, int64_t d_in, int epochs, int64_t batch, const pd_adamw &opt, int cosine, __half *v_out,
                           int32_t *axis_out, float *val_loss, unsigned char *scratch, uint32_t *status, cudaStream_t stream) {
    const int64_t m_max = batch > m_val ? batch : m_val;
    unsigned char *p = scratch + fit_scratch_bytes(m_max, d_out, d_in);
    uint32_t *mask_t = reinterpret_cast<uint32_t *>(p);
    p += round_up(static_cast<size_t>(d_in) * ((d_out + 31) / 32) * 4, 256);
    float *state = reinterpret_cast<float *>(p);
    p += round_up(static_cast<size_t>(4 * (d_out + d_in)) * 4, 256);
    float *train_loss = reinterpret_cast<float *>(p);
    pd_status st = launch_transpose_mask(mask, d_out, d_in, mask_t, stream);
    if (st != PD_OK) return st;
    const int64_t steps_per_epoch = (m_tr + batch - 1) / batch, total = steps_per_epoch * epochs;
    float *v_axis[2] = {state, state + 4 * d_out};
    for (int pass = 0; pass < 2; ++pass) {
        const int axis = pass == 0 ? PD_AXIS_COL : PD_AXIS_ROW;
        const int64_t len = axis == PD_AXIS_ROW ? d_out : d_in;
        float *v = v_axis[axis], *m1 = v + len, *m2 = m1 + len, *g = m2 + len;
        fit_init_kernel<<<static_cast<unsigned>((len + 255) / 256), 256, 0, stream>>>(axis == PD_AXIS_ROW ? v_row0 : v_col0, v, m1, m2,
                                                                                      static_cast<int>(len));
        count_launch();
        int64_t t = 0;
        for (int e = 0; e < epochs; ++e)
            for (int64_t b0 = 0; b0 < m_tr; b0 += batch) {
                const int64_t mb = m_tr - b0 < batch ? m_tr - b0 : batch;
                const double sched = cosine ? 0.5 * (1.0 + cos(3.14159265358979323846 * static_cast<double>(t) / static_cast<double>(total))) : 1.0;
                ++t;
                st = launch_fit_loss_grad(x_tr + b0 * d_in, y_tr + b0 * d_out, mb, w_b, mask, mask_t, v, axis, d_out, d_in, train_loss, g,
                                          scratch, status, stream);
                if (st != PD_OK) return st;
                st = launch_fit_adamw(v, m1, m2, g, len, t, static_cast<float>(opt.lr * sched), opt.beta1, opt.beta2, opt.eps,
                                      opt.weight_decay, nullptr, stream);
                if (st != PD_OK) return st;
            }
        st = launch_fit_loss_grad(x_val, y_val, m_val, w_b, mask, mask_t, v, axis, d_out, d_in, val_loss + axis, nullptr, scratch, status,
                                  stream);
        if (st != PD_OK) return st;
    }
    fit_select_kernel<<<32, 256, 0, stream>>>(val_loss, v_axis[PD_AXIS_ROW], static_cast<int>(d_out), v_axis[PD_AXIS_COL],
                                              static_cast<int>(d_in), v_out, axis_out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace pd
