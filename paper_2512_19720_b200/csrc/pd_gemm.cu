// Prefill path: Y[M, d_out] = X . (W_b + v (.) B)^T on the 5th-generation tensor cores.
//
// Two kernels share this file: gemm_pair_kernel (further down: tiles of 256 output rows on pairs of CTAs with
// tcgen05.mma.cta_group::2; every layer with at least 256 output rows) and gemm_kernel (one CTA per tile of 128 rows,
// described first; smaller layers).  Both form W_hat in tensor memory:
//
// The MMA computes the transposed tile  D[128 output rows, BN tokens] = W_hat_tile . X_tile^T :
//   A operand = W_hat tile, 128 rows x 64 k, in TENSOR MEMORY (row = lane, two fp16 per 32-bit column)
//   B operand = X tile, BN tokens x 64 k, K-major, 128-byte swizzle, in shared memory
//   D         = fp32 accumulator in tensor memory (256 columns)
// Putting the weights on the 128-row side means each W_b tile is expanded once per BN = 256
// tokens, the largest reuse one CTA can get.  Shared-memory bandwidth (TMA fills, LSU reads and
// tensor-core operand reads share one 128 B/clk pipe) is the scarce resource: forming W_hat in
// shared memory costs a write and a second read of every tile, forming it in tensor memory costs
// neither.
//
// Three rings per 64-wide k step, decoupled so that the weights can run ahead of the MMA:
//   x ring   (4..8 slots, shared memory)  warp 0 : TMA load of the x tile, signalled on ready[it % 8]
//   W_b ring (4..8 x 16 KB shared memory) warp 14: TMA load (+ the 64 col-axis scales) -> w_full[s];
//                                         freed by the transform warps once the tile row is in TMEM
//   W_hat ring (8 x 32 TMEM columns)      transform warps: W_b row from shared memory, +-v per mask bit
//                                         (mask words from global memory), tcgen05.st, arrive on ready[it % 8]
//   MMA warp        : ONE wait per k step (ready: x landed and W_hat written), four tcgen05.mma (K = 16 each)
//                     with A from TMEM, ONE tcgen05.commit -> consumed[it % 8], which frees the x slot (producer)
//                     and the W_hat slot (transform warps).  The issuing thread costs ~70 clocks per MMA or commit
//                     and ~100 per wait; with two waits and two commits it was slower than the tensor core.
//   epilogue warps  : wait acc_full; tcgen05.ld, fp16, shared-memory staging, 16-byte stores to y
// A thread of a transform warp owns one row of the tile (its TMEM lane) and all 64 k of a step; four
// warps take the even steps, four the odd ones.
// Every wait is bounded; a wait that runs out latches PD_ERR_DEVICE_TIMEOUT and the CTA
// drains and exits.
#include "pd_tcgen05.cuh"

namespace pd {
namespace {

constexpr int BM = 128;          // output rows per tile (MMA M)
constexpr int BK = 64;           // k per stage: 128 bytes of fp16 = one swizzle atom
constexpr int kMaxStages = 8;      // the x ring has SmemLayout<BN>::kXStages slots, the W_b ring ::kWStages
constexpr int kASlots = 8;        // W_hat ring (tensor memory, 32 columns each)
constexpr int kAccCols = 256;    // TMEM columns of the accumulator (one buffer)
constexpr int kAccBufs = 1;
constexpr int kACol0 = kAccBufs * kAccCols;  // first TMEM column of the W_hat ring: kASlots slots of 32 columns
constexpr int kVSlotBytes = 128;             // col axis: the 64 scales of a k step
constexpr int kNumWarps = 15;    // 0 x producer, 1 MMA, 2-5 epilogue, 6-13 transform, 14 W_b producer
constexpr int kNumThreads = kNumWarps * 32;
constexpr int kXformWarps = 8;
constexpr int kEpiWarps = 4;

struct GemmArgs {
    const uint32_t *mask;  // [d_out, d_in/32] or nullptr (base only)
    const __half *v;
    __half *y;
    int64_t ldy;
    int M, d_out, d_in;
    int tiles_m, tiles_n, k_steps;
    uint32_t *status;
    // grouped (multi-variant) mode: the token rows of x are already sorted by variant; token tile i is
    // tile_table[i] = {variant, first sorted row, rows, 0}; variant V means "base only"
    const int4 *tile_table;
    const int *n_token_tiles;   // device: number of entries of tile_table
    const int *row_index;       // sorted row -> row of y
    int64_t mask_stride, v_stride;  // elements between two variants' masks / scale vectors
    unsigned long long col_axis_bits;  // bit g set: variant g scales along d_in
    int V;
    int y_vec_ok;  // y is 16-byte aligned and ldy a multiple of 8: rows can be written with 16-byte stores
    int token_tile;  // pair kernel, one variant: tokens per tile (64, 128 or 256)
    int bf16;        // host side only: which instantiation to launch
    // pair kernel, one variant: the k steps are dealt to `splits` tiles (k_steps counts one split's steps); with
    // splits > 1 a tile writes its fp32 partial sums to partial[split][token][row] and splitk_reduce_kernel adds them
    int splits;
    float *partial;
};

struct Tile {
    int tm, tok0, count;    // W row tile; first token row (of x); valid tokens
    const uint32_t *mask;
    const __half *v;
    bool col, delta;
};

template <int AXIS, bool HAS_DELTA, bool GROUPED, int BN>
__device__ __forceinline__ Tile get_tile(const GemmArgs &a, int tile, int n_tt) {
    Tile t;
    t.tm = tile / n_tt;
    const int tn = tile - t.tm * n_tt;
    if (!GROUPED) {
        t.tok0 = tn * BN;
        t.count = min(BN, a.M - t.tok0);
        t.mask = a.mask;
        t.v = a.v;
        t.col = AXIS == PD_AXIS_COL;
        t.delta = HAS_DELTA;
    } else {
        const int4 e = __ldg(a.tile_table + tn);
        t.tok0 = e.y;
        t.count = e.z;
        t.delta = e.x < a.V;
        const int g = t.delta ? e.x : 0;
        t.mask = a.mask + static_cast<size_t>(g) * a.mask_stride;
        t.v = a.v + static_cast<size_t>(g) * a.v_stride;
        t.col = (a.col_axis_bits >> g) & 1ull;
    }
    return t;
}


template <int BN>
struct SmemLayout {
    static constexpr int kWBytes = BM * BK * 2;   // 16 KB
    static constexpr int kXBytes = BN * BK * 2;   // 32 KB for BN = 256
    static constexpr int kXOffset = 0;                       // x ring
    // W_b ring: what a narrow x tile leaves free goes to more W_b stages -- with few tokens per tile a k step is
    // short and only a deep ring hides the L2/HBM latency of the weight tiles
    static constexpr int kWStages = BN == 256 ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int kXStages = kWStages;
    static constexpr int kWOffset = kXStages * kXBytes;
    static constexpr int kBarOffset = kWOffset + kWStages * kWBytes;
    static constexpr int kVOffset = kBarOffset + 512;        // kWStages slots of kVSlotBytes
    static constexpr int kOutOffset = kVOffset + kWStages * kVSlotBytes;   // epilogue staging: [128 tokens][128 rows] fp16
    static_assert(kWStages % 2 == 0 && kWStages <= kMaxStages, "even and odd k steps belong to different warps");
    static constexpr int kTotal = kOutOffset + 128 * 128 * 2 + 1024;      // + slack for 1024-byte alignment
};

// One row of a W_hat tile: 64 columns = 8 pieces of 16 bytes read from the 128-byte-swizzled W_b tile, +-v added
// per mask bit (word0 = columns 0..31, word1 = columns 32..63), packed two fp16 per register in column order.
template <bool BF16, bool DELTA, bool COL>
__device__ __forceinline__ void build_w_hat_row(uint32_t (&out)[32], const unsigned char *wt, const unsigned char *vs, int r,
                                                uint32_t vrow, uint32_t word0, uint32_t word1) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {  // 16-byte piece c = columns 8c .. 8c+7 of the stage
        const uint4 w = *reinterpret_cast<const uint4 *>(wt + ((c ^ (r & 7)) << 4));
        const uint32_t wp[4] = {w.x, w.y, w.z, w.w};
        if (DELTA) {
            uint32_t vv[4] = {vrow, vrow, vrow, vrow};
            if (COL) {
                const uint4 t4 = *reinterpret_cast<const uint4 *>(vs + 16 * c);
                vv[0] = t4.x, vv[1] = t4.y, vv[2] = t4.z, vv[3] = t4.w;
                if (BF16) {  // the scales arrive as binary16: one rounding to the weights' type
#pragma unroll
                    for (int pr = 0; pr < 4; ++pr) vv[pr] = Elem<BF16>::scale_pair2(vv[pr]);
                }
            }
            // the piece's 8 sign bits are byte c & 3 of its word.  b * 0x8001 puts bit i at i and i + 15, so a left
            // shift by 15 - 2 pr brings bit 2 pr to bit 15 and bit 2 pr + 1 to bit 31: the signs of halves 2 pr (low)
            // and 2 pr + 1 (high).  +v where the bit is 1, -v where it is 0.
            const uint32_t sp = prmt(c < 4 ? word0 : word1, 0u, 0x4440u | static_cast<uint32_t>(c & 3)) * 0x8001u;
#pragma unroll
            for (int pr = 0; pr < 4; ++pr)
                out[4 * c + pr] = Elem<BF16>::add2(wp[pr], lop3_andn_xor(sp << (15 - 2 * pr), 0x80008000u, vv[pr]));
        } else {  // base only: the tile goes to tensor memory unchanged
#pragma unroll
            for (int pr = 0; pr < 4; ++pr) out[4 * c + pr] = wp[pr];
        }
    }
}

template <bool BF16, int AXIS, bool HAS_DELTA, bool GROUPED, int BN>
__global__ void __launch_bounds__(kNumThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const GemmArgs a) {
    using L = SmemLayout<BN>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBarOffset);
    // ready[it % 8]   : k step `it` can be multiplied -- its x tile has landed (TMA bytes + the producer's arrival)
    //                   and its W_hat slot is written (four transform warps);
    // consumed[it % 8]: the MMAs of k step `it` have finished reading both (tcgen05.commit).
    // One wait and one commit per k step keep the single MMA-issuing thread ahead of the tensor core.
    uint64_t *w_full = bars, *w_empty = bars + kMaxStages;
    uint64_t *ready = bars + 2 * kMaxStages, *consumed = ready + kASlots;
    uint64_t *acc_full = consumed + kASlots, *acc_empty = acc_full + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 1);
    static_assert((2 * kMaxStages + 2 * kASlots + 2) * 8 + 8 <= 512, "barrier block");
    static_assert(L::kXStages <= kASlots, "an x slot must be free again before its ready barrier comes round");
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tt = GROUPED ? __ldg(a.n_token_tiles) : a.tiles_n;  // token tiles
    const int n_tiles = a.tiles_m * n_tt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < L::kWStages; ++s) {
            mbar_init(w_full + s, 1);
            mbar_init(w_empty + s, kXformWarps / 2);  // the four warps (one per TMEM lane quarter) that own the stage
        }
        for (int s = 0; s < kASlots; ++s) {
            mbar_init(ready + s, kXformWarps / 2 + 1);
            mbar_init(consumed + s, 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(acc_full + b, 1);
            mbar_init(acc_empty + b, kEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < L::kWStages * kVSlotBytes / 4) {  // scale slots start at zero: a short last k step leaves its tail untouched
        reinterpret_cast<uint32_t *>(smem + L::kVOffset)[threadIdx.x] = 0u;
        fence_proxy_async_smem();
    }
    if (warp == 1) tcgen05_alloc(tmem_slot, 512);
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0 || warp == kNumWarps - 1) {
        // ------------------------------------------------ TMA producers: warp 0 feeds the x ring, the last warp the W_b ring
        if (lane == 0) {
            const bool is_x = warp == 0;
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const Tile ti = get_tile<AXIS, HAS_DELTA, GROUPED, BN>(a, tile, n_tt);
                for (int ks = 0; ks < a.k_steps; ++ks, ++it) {
                    const int ring = is_x ? L::kXStages : L::kWStages;
                    const int s = it % ring;
                    const uint32_t parity = ((it / ring) & 1) ^ 1;
                    if (is_x) {
                        // the x slot was last read by k step it - kXStages
                        if (it >= static_cast<uint32_t>(L::kXStages)) {
                            const uint32_t prev = it - L::kXStages;
                            if (!(ok = mbar_wait(consumed + prev % kASlots, (prev / kASlots) & 1, abort_flag, a.status, 1))) break;
                        }
                        mbar_arrive_expect_tx(ready + it % kASlots, L::kXBytes);
                        tma_load_2d(&map_x, ready + it % kASlots, smem + L::kXOffset + s * L::kXBytes, ks * BK, ti.tok0);
                    } else {
                        if (!(ok = mbar_wait(w_empty + s, parity, abort_flag, a.status, 6))) break;
                        const uint32_t v_bytes = (ti.delta && ti.col) ? static_cast<uint32_t>(min(BK, a.d_in - ks * BK) * 2) : 0u;
                        mbar_arrive_expect_tx(w_full + s, L::kWBytes + v_bytes);
                        tma_load_2d(&map_w, w_full + s, smem + L::kWOffset + s * L::kWBytes, ks * BK, ti.tm * BM);
                        if (v_bytes) bulk_load_1d(smem + L::kVOffset + s * kVSlotBytes, ti.v + static_cast<size_t>(ks) * BK, v_bytes, w_full + s);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer: A = W_hat slot in tensor memory, B = x tile in shared memory
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tcount) {
                // MMA N = the tile's tokens rounded up to 16 (the whole token box in the plain mode)
                const Tile ti = get_tile<AXIS, HAS_DELTA, GROUPED, BN>(a, tile, n_tt);
                const int n_mma = GROUPED ? ((ti.count + 15) & ~15) : BN;
                const uint32_t idesc = kIdescBase<BF16> | (static_cast<uint32_t>(n_mma >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);
                const uint32_t b = tcount % kAccBufs;
                if (!(ok = mbar_wait(acc_empty + b, ((tcount / kAccBufs) & 1) ^ 1, abort_flag, a.status, 2))) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + b * kAccCols;
                for (int ks = 0; ks < a.k_steps; ++ks, ++it) {
                    const int s = it % L::kXStages, sa = it % kASlots;
                    if (!(ok = mbar_wait(ready + sa, (it / kASlots) & 1, abort_flag, a.status, 3))) break;
                    tcgen05_fence_after();
                    const uint32_t x_addr = smem_u32(smem + L::kXOffset + s * L::kXBytes);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)
                        tcgen05_mma_f16_tmem_a(d_tmem, tmem_base + kACol0 + sa * 32 + kk * 8, make_smem_desc(x_addr + kk * 32), idesc,
                                               (ks > 0 || kk > 0) ? 1u : 0u);
                    tcgen05_commit(consumed + sa);  // the x slot and the W_hat slot free up when these MMAs have read them
                }
                if (ok) tcgen05_commit(acc_full + b);
            }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ------------------------------------------------ epilogue: TMEM -> fp16 -> shared-memory staging -> y[token][row]
        // The accumulator is drained in two halves of 128 tokens through a 32 KB staging tile laid out
        // [token][128 rows], so that y is written with 16-byte stores, 256 contiguous bytes per token; the
        // accumulator is handed back to the MMA warp as soon as its last column has been read.
        const int quarter = warp & 3;  // the 32 TMEM lanes this warp may read
        const int et = threadIdx.x - 2 * 32;  // 0..127 among the epilogue threads
        unsigned char *stage_out = smem + L::kOutOffset;
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tcount) {
            const Tile ti = get_tile<AXIS, HAS_DELTA, GROUPED, BN>(a, tile, n_tt);
            const uint32_t b = tcount % kAccBufs;
            const bool got = mbar_wait(acc_full + b, (tcount / kAccBufs) & 1, abort_flag, a.status, 4);
            uint32_t gave_up;  // OR over the four epilogue warps, so that they leave together
            asm volatile(
                "{\n"
                ".reg .pred p, q;\n"
                "setp.ne.u32 q, %1, 0;\n"
                "bar.red.or.pred p, 2, %2, q;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(gave_up)
                : "r"(static_cast<uint32_t>(!got)), "n"(kEpiWarps * 32)
                : "memory");
            if (gave_up) break;
            tcgen05_fence_after();
            const int row_l = quarter * 32 + lane;          // row of the tile this thread reads from TMEM
            const int o0 = ti.tm * BM;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + b * kAccCols;
            const int n_half = (ti.count + 127) / 128;      // 1 or 2
            for (int hf = 0; hf < n_half; ++hf) {
#pragma unroll 1
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    if (hf * 128 + c0 >= ti.count) break;  // warp-uniform: no token of this tile lives in these columns
                    uint32_t r[32];
                    tcgen05_ld_32x32b_x32(taddr + hf * 128 + c0, r);
                    tcgen05_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        *reinterpret_cast<unsigned short *>(stage_out + (c0 + j) * 256 + row_l * 2) = Elem<BF16>::from_float(__uint_as_float(r[j]));
                }
                if (hf == n_half - 1) {  // every column of the accumulator has been read
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty + b);
                }
                asm volatile("bar.sync 2, %0;" ::"n"(kEpiWarps * 32) : "memory");
                const int n_tok = min(128, ti.count - hf * 128);
                for (int idx = et; idx < n_tok * 16; idx += kEpiWarps * 32) {
                    const int tok = idx >> 4, ch = idx & 15;
                    const int yr = GROUPED ? __ldg(a.row_index + ti.tok0 + hf * 128 + tok) : ti.tok0 + hf * 128 + tok;
                    const int o = o0 + ch * 8;
                    __half *dst = a.y + static_cast<size_t>(yr) * a.ldy + o;
                    const uint4 val = *reinterpret_cast<const uint4 *>(stage_out + tok * 256 + ch * 16);
                    if (a.y_vec_ok && o + 8 <= a.d_out) {
                        *reinterpret_cast<uint4 *>(dst) = val;
                    } else {
                        const __half *hv = reinterpret_cast<const __half *>(&val);
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            if (o + q < a.d_out) dst[q] = hv[q];
                    }
                }
                asm volatile("bar.sync 2, %0;" ::"n"(kEpiWarps * 32) : "memory");
            }
        }
    } else {
        // ------------------------------------------------ transform: W_b tile (shared memory) -> W_hat slot (tensor memory)
        // A thread owns one row of the tile (its TMEM lane) and all 64 k of a stage; the four warps with
        // (warp - 6) / 4 == 0 take the even stages, the other four the odd ones.
        const int quarter = warp & 3;                 // the 32 TMEM lanes this warp may write
        const uint32_t par = static_cast<uint32_t>((warp - (2 + kEpiWarps)) >> 2);
        const int r = quarter * 32 + lane;            // tile row
        const int words = a.d_in >> 5;
        const uint32_t a_taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + kACol0;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            const Tile ti = get_tile<AXIS, HAS_DELTA, GROUPED, BN>(a, tile, n_tt);
            const bool delta = ti.delta, col = ti.col;  // compile-time constants in the plain mode
            const int o = ti.tm * BM + r;
            const bool row_ok = o < a.d_out;
            uint32_t vrow = 0;
            if (delta && !col && row_ok) {
                vrow = Elem<BF16>::scale_pair(*reinterpret_cast<const unsigned short *>(ti.v + o));
            }
            const uint32_t *mrow = delta ? ti.mask + static_cast<size_t>(row_ok ? o : 0) * words : nullptr;
            auto load_words = [&](int ks, uint32_t &w0, uint32_t &w1) {
                w0 = (delta && row_ok && ks < a.k_steps && 2 * ks < words) ? __ldg(mrow + 2 * ks) : 0u;
                w1 = (delta && row_ok && ks < a.k_steps && 2 * ks + 1 < words) ? __ldg(mrow + 2 * ks + 1) : 0u;
            };
            int ks = static_cast<int>((par ^ it) & 1u);  // first k step of this tile that falls to this warp
            // mask words of the next four k steps of this warp, in flight: they come from L2 or HBM, and with few
            // tokens per tile a k step is far shorter than that latency
            uint32_t q0[4], q1[4];
#pragma unroll
            for (int d = 0; d < 4; ++d) load_words(ks + 2 * d, q0[d], q1[d]);
            for (; ks < a.k_steps; ks += 2) {
                const uint32_t my_it = it + ks;
                const int s = my_it % L::kWStages, sa = my_it % kASlots;
                const uint32_t word[2] = {q0[0], q1[0]};
#pragma unroll
                for (int d = 0; d < 3; ++d) q0[d] = q0[d + 1], q1[d] = q1[d + 1];
                load_words(ks + 8, q0[3], q1[3]);
                // the TMEM store below is warp-collective: all lanes leave together or not at all
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(w_full + s, (my_it / L::kWStages) & 1, abort_flag, a.status, 5)))) break;
                const unsigned char *wt = smem + L::kWOffset + s * L::kWBytes + r * 128;
                const unsigned char *vs = smem + L::kVOffset + s * kVSlotBytes;
                uint32_t out[32];
                // specialised bodies: with the variant known only at run time (grouped mode) a single body with
                // the tests inside the unrolled loop spilled registers and ran four times slower
                if (!delta) build_w_hat_row<BF16, false, false>(out, wt, vs, r, vrow, word[0], word[1]);
                else if (col) build_w_hat_row<BF16, true, true>(out, wt, vs, r, vrow, word[0], word[1]);
                else build_w_hat_row<BF16, true, false>(out, wt, vs, r, vrow, word[0], word[1]);
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(consumed + sa, ((my_it / kASlots) & 1) ^ 1, abort_flag, a.status, 8)))) break;
                tcgen05_fence_after();
                tcgen05_st_32x32b_x32(a_taddr + sa * 32, out);
                // The store takes every register of the tile row as an operand, so all shared-memory reads of the
                // W_b slot have returned by now: only here may the slot be handed back for refilling.
                __syncwarp();
                if (lane == 0) mbar_arrive(w_empty + s);
                tcgen05_wait_st();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(ready + sa);
            }
            it += a.k_steps;
        }
    }

    // ------------------------------------------------ teardown
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait ran out somewhere: give copies that may still be in flight time to land
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------ CTA-pair kernel (M >= 256, one variant)
//
// Two CTAs of a cluster (two SMs) work on one tile of 256 output rows x 256 tokens with
// tcgen05.mma.cta_group::2: each CTA expands its own 128 rows of W_hat into its own tensor memory and
// holds only HALF of the x tile (128 tokens) in shared memory; the tensor cores of both SMs read both
// halves.  Per k step a CTA therefore moves 16 KB of x instead of 32 KB through shared memory, twice
// (TMA fill, operand read): shared-memory bandwidth, which caps the one-CTA kernel at about two thirds
// of the tensor peak, is no longer the limit.
//
// Rank 0 of the pair issues every MMA: per TWO k steps one wait, eight MMAs and one commit (a wait costs the
// issuing thread ~110 clocks, a commit ~70, an MMA ~70 against 128 clocks of tensor work: per single k step the
// thread was the bottleneck).  The k steps of a tile are rounded up to an even number; a step past d_in reads
// zeros.  Barriers that gate the MMA thread live in rank 0 only:
//   ready[pair % 4] : 4 transform warps of each CTA for each of the two steps (rank 1 arrives remotely) + rank 0's
//                     x producer, which also announces the bytes of BOTH x halves of both steps; rank 1's TMA
//                     reports its bytes to rank 0's barrier
//   acc_empty       : the 4 epilogue warps of each CTA
// consumed[] and acc_full exist in both CTAs; one multicast tcgen05.commit arrives on both copies.
// The W_b ring, its barriers and the transform are per CTA, as in the kernel above.
constexpr int kPairSlots = kASlots / 2;  // ready / consumed barriers: one per two k steps
// warps: 0 x producer, 1 MMA, then the epilogue warps, 8 transform warps, the W_b producer.  Eight epilogue warps
// for full tiles of 256 tokens; the multi-variant tiles are narrower and the four warps saved leave the
// transform 128 registers per thread instead of 96.
__host__ __device__ constexpr int pair_epi_warps(bool grouped) { return grouped ? 4 : 8; }
__host__ __device__ constexpr int pair_threads(bool grouped) { return (2 + pair_epi_warps(grouped) + kXformWarps + 1) * 32; }
struct PairLayout {
    static constexpr int kStages = 6;             // x ring and W_b ring
    static constexpr int kWBytes = BM * BK * 2;   // 16 KB
    static constexpr int kXBytes = 128 * BK * 2;  // this CTA's half of the token tile: 16 KB
    static constexpr int kXOffset = 0;
    static constexpr int kWOffset = kStages * kXBytes;
    static constexpr int kBarOffset = kWOffset + kStages * kWBytes;
    static constexpr int kVOffset = kBarOffset + 512;
    static constexpr int kOutOffset = kVOffset + kStages * kVSlotBytes;
    static constexpr int kTotal = kOutOffset + 128 * 128 * 2 + 1024;
    // A W_b stage must always fall to the same transform group (even / odd k steps).  Were stages dealt to the
    // groups in turn, a group could wait for "its" phase of a stage while the other group's phase of that stage is
    // still in flight, see the parity of the phase before that one and take the stage too early.
    static_assert(kStages % 2 == 0 && kStages <= kASlots, "ring depth");
    static_assert(kTotal <= 227 * 1024, "shared memory per CTA");
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of `p` (a shared-memory object of this CTA) in the CTA of the given rank
__device__ __forceinline__ uint32_t map_to_rank(const void *p, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The waits on barriers that the other CTA arrives on are the plain mbar_wait: the operands the MMA reads travel
// through the async proxy (TMA, tcgen05.st + fences), and cluster-scoped acquire/release qualifiers on the per-step
// barrier operations cost 30 % of the kernel's throughput.

// x half of this CTA; the bytes are reported to the barrier at `bar_cluster_addr` (rank 0's)
__device__ __forceinline__ void tma_load_2d_pair(const CUtensorMap *map, uint32_t bar_cluster_addr, void *dst, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tcgen05_alloc_pair(uint32_t *dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// arrives on the barrier at the same offset in both CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void tcgen05_commit_pair(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                     smem_u32(bar)),
                 "h"(static_cast<unsigned short>(3))
                 : "memory");
}
__device__ __forceinline__ void tcgen05_mma_f16_tmem_a_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                            uint32_t accumulate) {
    const uint32_t z = 0;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n"
        "}\n" ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z)
        : "memory");
}

// Tile of the pair kernel as one CTA sees it.  `half` = token rows each CTA holds in shared memory (MMA N = 2 half).
struct PairTile {
    int tm, tok0, count, half;   // this CTA's W row tile of 128; first token row; valid tokens; tokens per CTA
    int k0, split;               // first k step of the tile (split-K), and which split it is
    const uint32_t *mask;
    const __half *v;
    bool col, delta;
};
template <int AXIS, bool HAS_DELTA, bool GROUPED>
__device__ __forceinline__ PairTile get_pair_tile(const GemmArgs &a, int tile, int n_tt, uint32_t rank) {
    PairTile t;
    t.k0 = 0, t.split = 0;
    if (!GROUPED && a.splits > 1) {  // the splits of one output tile are neighbours: they share the x tile and finish together
        t.split = tile % a.splits;
        tile /= a.splits;
        t.k0 = t.split * a.k_steps;
    }
    const int tp = tile / n_tt, tn = tile - tp * n_tt;
    t.tm = 2 * tp + static_cast<int>(rank);
    if (!GROUPED) {  // MMA N = the tile's tokens rounded up to a multiple of 32
        t.tok0 = tn * a.token_tile;
        t.count = min(a.token_tile, a.M - t.tok0);
        t.half = ((t.count + 31) & ~31) >> 1;
        t.mask = a.mask;
        t.v = a.v;
        t.col = AXIS == PD_AXIS_COL;
        t.delta = HAS_DELTA;
    } else {  // one variant's rows (at most 256), MMA N rounded up to a multiple of 32
        const int4 e = __ldg(a.tile_table + tn);
        t.tok0 = e.y;
        t.count = e.z;
        t.half = ((e.z + 31) & ~31) >> 1;
        t.delta = e.x < a.V;
        const int g = t.delta ? e.x : 0;
        t.mask = a.mask + static_cast<size_t>(g) * a.mask_stride;
        t.v = a.v + static_cast<size_t>(g) * a.v_stride;
        t.col = (a.col_axis_bits >> g) & 1ull;
    }
    return t;
}

template <bool BF16, int AXIS, bool HAS_DELTA, bool GROUPED>
__global__ void __launch_bounds__(pair_threads(GROUPED), 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const GemmArgs a) {
    using L = PairLayout;
    constexpr int kEpiW = pair_epi_warps(GROUPED), kWarps = pair_threads(GROUPED) / 32;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::kBarOffset);
    uint64_t *w_full = bars, *w_empty = bars + kMaxStages;
    uint64_t *ready = bars + 2 * kMaxStages, *consumed = ready + kASlots;
    uint64_t *acc_full = consumed + kASlots, *acc_empty = acc_full + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 issues the MMAs
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int tiles_m2 = (a.tiles_m + 1) >> 1;        // tiles of 256 rows
    const int n_tt = GROUPED ? __ldg(a.n_token_tiles) : a.tiles_n;  // token tiles
    const int n_tiles = tiles_m2 * n_tt * (GROUPED ? 1 : a.splits);

    if (threadIdx.x == 0) {
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(w_full + s, 1);
            mbar_init(w_empty + s, kXformWarps / 2);
        }
        for (int s = 0; s < kASlots; ++s) {
            mbar_init(ready + s, 2 * kXformWarps + 1);  // used in rank 0 only: two k steps x two CTAs x four warps + x
            mbar_init(consumed + s, 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 2 * kEpiW);               // used in rank 0 only
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < L::kStages * kVSlotBytes / 4) {
        reinterpret_cast<uint32_t *>(smem + L::kVOffset)[threadIdx.x] = 0u;
        fence_proxy_async_smem();
    }
    if (warp == 1) tcgen05_alloc_pair(tmem_slot, 512);
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();  // the other CTA's barriers are initialised before anything arrives on them
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    auto tile_of = [&](int tile) { return get_pair_tile<AXIS, HAS_DELTA, GROUPED>(a, tile, n_tt, rank); };

    if (warp == 0 || warp == kWarps - 1) {
        // ------------------------------------------------ TMA producers
        if (lane == 0) {
            const bool is_x = warp == 0;
            uint32_t it = 0;
            bool ok = true;
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
                const PairTile ti = tile_of(tile);
                for (int ks = 0; ks < a.k_steps; ++ks, ++it) {
                    const int s = it % L::kStages;
                    if (is_x) {
                        const uint32_t pi = it >> 1;  // pair of k steps: one ready / consumed barrier for both
                        if ((it & 1u) == 0) {
                            if (pi >= static_cast<uint32_t>(L::kStages / 2)) {  // the two x slots were last read by pair pi - 3
                                const uint32_t prev = pi - L::kStages / 2;
                                if (!(ok = mbar_wait(consumed + prev % kPairSlots, (prev / kPairSlots) & 1, abort_flag, a.status, 1))) break;
                            }
                            if (rank == 0) mbar_arrive_expect_tx(ready + pi % kPairSlots, 4 * L::kXBytes);  // both halves of both steps
                        }
                        tma_load_2d_pair(&map_x, map_to_rank(ready + pi % kPairSlots, 0), smem + L::kXOffset + s * L::kXBytes,
                                         (ti.k0 + ks) * BK, ti.tok0 + ti.half * static_cast<int>(rank));
                    } else {
                        const uint32_t parity = ((it / L::kStages) & 1) ^ 1;
                        if (!(ok = mbar_wait(w_empty + s, parity, abort_flag, a.status, 6))) break;
                        const int ka = ti.k0 + ks;
                        const uint32_t v_bytes = (ti.delta && ti.col) ? static_cast<uint32_t>(max(0, min(BK, a.d_in - ka * BK)) * 2) : 0u;
                        mbar_arrive_expect_tx(w_full + s, L::kWBytes + v_bytes);
                        tma_load_2d(&map_w, w_full + s, smem + L::kWOffset + s * L::kWBytes, ka * BK, ti.tm * BM);
                        if (v_bytes) bulk_load_1d(smem + L::kVOffset + s * kVSlotBytes, ti.v + static_cast<size_t>(ka) * BK, v_bytes, w_full + s);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (rank 0 only): M = 256 over both CTAs, N = 256
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++tcount) {
                const int n_mma = 2 * tile_of(tile).half;
                const uint32_t idesc = kIdescBase<BF16> | (static_cast<uint32_t>(n_mma >> 3) << 17) | (static_cast<uint32_t>(256 >> 4) << 24);
                if (!(ok = mbar_wait(acc_empty, (tcount & 1) ^ 1, abort_flag, a.status, 2))) break;
                tcgen05_fence_after();
                for (int ks = 0; ks < a.k_steps; ks += 2, it += 2) {
                    const uint32_t pi = it >> 1;
                    if (!(ok = mbar_wait(ready + pi % kPairSlots, (pi / kPairSlots) & 1, abort_flag, a.status, 3))) break;
                    tcgen05_fence_after();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t x_addr = smem_u32(smem + L::kXOffset + ((it + h) % L::kStages) * L::kXBytes);
                        const uint32_t a_col = tmem_base + kACol0 + ((it + h) % kASlots) * 32;
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk)
                            tcgen05_mma_f16_tmem_a_pair(tmem_base, a_col + kk * 8, make_smem_desc(x_addr + kk * 32), idesc,
                                                        (ks > 0 || h > 0 || kk > 0) ? 1u : 0u);
                    }
                    tcgen05_commit_pair(consumed + pi % kPairSlots);  // frees the x slots and the W_hat slots of both steps
                }
                if (ok) tcgen05_commit_pair(acc_full);
            }
        }
    } else if (warp < 2 + kEpiW) {
        // ------------------------------------------------ epilogue: this CTA's 128 rows of the accumulator, as in the kernel above
        // eight warps: two per TMEM lane quarter, each draining half of the columns, so that the accumulator goes
        // back to the MMA thread in half the time (the tensor cores idle while it is drained)
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;
        constexpr int kColsPerWarp = 128 / (kEpiW / 4);  // of each half of 128 tokens
        const int et = threadIdx.x - 2 * 32;
        unsigned char *stage_out = smem + L::kOutOffset;
        const uint32_t acc_empty_rank0 = map_to_rank(acc_empty, 0);
        uint32_t tcount = 0;
        for (int tile = pair; tile < n_tiles; tile += n_pairs, ++tcount) {
            const PairTile ti = tile_of(tile);
            const int tok0 = ti.tok0, count = ti.count;
            const bool got = mbar_wait(acc_full, tcount & 1, abort_flag, a.status, 4);
            uint32_t gave_up;  // OR over the four epilogue warps, so that they leave together
            asm volatile(
                "{\n"
                ".reg .pred p, q;\n"
                "setp.ne.u32 q, %1, 0;\n"
                "bar.red.or.pred p, 2, %2, q;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(gave_up)
                : "r"(static_cast<uint32_t>(!got)), "n"(kEpiW * 32)
                : "memory");
            if (gave_up) break;
            tcgen05_fence_after();
            const int row_l = quarter * 32 + lane;
            const int o0 = ti.tm * BM;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const int n_half = (count + 127) / 128;
            if (!GROUPED && a.splits > 1) {
                // split-K: the fp32 partial sums go to partial[split][token][row]; a lane owns a row, so the 32 lanes of
                // a warp write 128 contiguous bytes per token
                const int o = o0 + row_l;
                float *dst = a.partial + (static_cast<size_t>(ti.split) * a.M + tok0) * a.d_out + o;
                for (int hf = 0; hf < n_half; ++hf) {
#pragma unroll 1
                    for (int c0 = kColsPerWarp * col_half; c0 < kColsPerWarp * (col_half + 1); c0 += 32) {
                        if (hf * 128 + c0 >= count) break;
                        uint32_t r[32];
                        tcgen05_ld_32x32b_x32(taddr + hf * 128 + c0, r);
                        tcgen05_wait_ld();
                        if (o < a.d_out) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (hf * 128 + c0 + j < count) dst[static_cast<size_t>(hf * 128 + c0 + j) * a.d_out] = __uint_as_float(r[j]);
                        }
                    }
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty_rank0);
                continue;
            }
            for (int hf = 0; hf < n_half; ++hf) {
#pragma unroll 1
                for (int c0 = kColsPerWarp * col_half; c0 < kColsPerWarp * (col_half + 1); c0 += 32) {
                    if (hf * 128 + c0 >= count) break;
                    uint32_t r[32];
                    tcgen05_ld_32x32b_x32(taddr + hf * 128 + c0, r);
                    tcgen05_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        *reinterpret_cast<unsigned short *>(stage_out + (c0 + j) * 256 + row_l * 2) = Elem<BF16>::from_float(__uint_as_float(r[j]));
                }
                if (hf == n_half - 1) {  // every column of the accumulator has been read
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty_rank0);
                }
                asm volatile("bar.sync 2, %0;" ::"n"(kEpiW * 32) : "memory");
                const int n_tok = min(128, count - hf * 128);
                for (int idx = et; idx < n_tok * 16; idx += kEpiW * 32) {
                    const int tok = idx >> 4, ch = idx & 15;
                    const int o = o0 + ch * 8;
                    const int yr = GROUPED ? __ldg(a.row_index + tok0 + hf * 128 + tok) : tok0 + hf * 128 + tok;
                    __half *dst = a.y + static_cast<size_t>(yr) * a.ldy + o;
                    const uint4 val = *reinterpret_cast<const uint4 *>(stage_out + tok * 256 + ch * 16);
                    if (a.y_vec_ok && o + 8 <= a.d_out) {
                        *reinterpret_cast<uint4 *>(dst) = val;
                    } else {
                        const __half *hv = reinterpret_cast<const __half *>(&val);
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            if (o + q < a.d_out) dst[q] = hv[q];
                    }
                }
                asm volatile("bar.sync 2, %0;" ::"n"(kEpiW * 32) : "memory");
            }
        }
    } else {
        // ------------------------------------------------ transform: this CTA's W_b tile -> its W_hat slot, as in the kernel above
        const int quarter = warp & 3;
        const uint32_t par = static_cast<uint32_t>((warp - (2 + kEpiW)) >> 2);
        const int r = quarter * 32 + lane;
        const int words = a.d_in >> 5;
        const uint32_t a_taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + kACol0;
        const uint32_t ready_rank0 = map_to_rank(ready, 0);
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
            const PairTile ti = tile_of(tile);
            const bool delta = ti.delta, col = ti.col;  // compile-time constants in the plain mode
            const int o = ti.tm * BM + r;
            const bool row_ok = o < a.d_out;
            uint32_t vrow = 0;
            if (delta && !col && row_ok) {
                vrow = Elem<BF16>::scale_pair(*reinterpret_cast<const unsigned short *>(ti.v + o));
            }
            const uint32_t *mrow = delta ? ti.mask + static_cast<size_t>(row_ok ? o : 0) * words : nullptr;
            const int k0 = ti.k0;
            auto load_words = [&](int ks, uint32_t &w0, uint32_t &w1) {
                w0 = (delta && row_ok && ks < a.k_steps && 2 * (k0 + ks) < words) ? __ldg(mrow + 2 * (k0 + ks)) : 0u;
                w1 = (delta && row_ok && ks < a.k_steps && 2 * (k0 + ks) + 1 < words) ? __ldg(mrow + 2 * (k0 + ks) + 1) : 0u;
            };
            int ks = static_cast<int>((par ^ it) & 1u);
            uint32_t q0[4], q1[4];
#pragma unroll
            for (int d = 0; d < 4; ++d) load_words(ks + 2 * d, q0[d], q1[d]);
            for (; ks < a.k_steps; ks += 2) {
                const uint32_t my_it = it + ks;
                const int s = my_it % L::kStages, sa = my_it % kASlots;
                const uint32_t word[2] = {q0[0], q1[0]};
#pragma unroll
                for (int d = 0; d < 3; ++d) q0[d] = q0[d + 1], q1[d] = q1[d + 1];
                load_words(ks + 8, q0[3], q1[3]);
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(w_full + s, (my_it / L::kStages) & 1, abort_flag, a.status, 5)))) break;
                const unsigned char *wt = smem + L::kWOffset + s * L::kWBytes + r * 128;
                const unsigned char *vs = smem + L::kVOffset + s * kVSlotBytes;
                uint32_t out[32];
                // specialised bodies: a single body with run-time tests inside the unrolled loop spills
                if (!delta) build_w_hat_row<BF16, false, false>(out, wt, vs, r, vrow, word[0], word[1]);
                else if (col) build_w_hat_row<BF16, true, true>(out, wt, vs, r, vrow, word[0], word[1]);
                else build_w_hat_row<BF16, true, false>(out, wt, vs, r, vrow, word[0], word[1]);
                const uint32_t pi = my_it >> 1;  // the W_hat slot was last read by pair pi - 4
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(consumed + pi % kPairSlots, ((pi / kPairSlots) & 1) ^ 1, abort_flag, a.status, 8)))) break;
                tcgen05_fence_after();
                tcgen05_st_32x32b_x32(a_taddr + sa * 32, out);
                // all shared-memory reads of the W_b slot have returned once the store has taken its operands
                __syncwarp();
                if (lane == 0) mbar_arrive(w_empty + s);
                tcgen05_wait_st();
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(ready_rank0 + (pi % kPairSlots) * 8u);
            }
            it += a.k_steps;
        }
    }

    // ------------------------------------------------ teardown: neither CTA may leave (or free tensor memory) while the
    // other can still read its shared memory, arrive on its barriers or multiply from its tensor memory
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
        __syncthreads();
    }
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tcgen05_fence_after();
        tcgen05_dealloc_pair(tmem_base, 512);
    }
}


// Split-K: y[token][row] = sum over the splits, in split order, of partial[split][token][row], rounded once to the
// storage type.  Four rows per thread.
template <bool BF16>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *partial, int splits, int M, int d_out, __half *y, int64_t ldy, int vec_ok) {
    asm volatile("griddepcontrol.wait;" ::: "memory");  // launched while the GEMM still runs
    const int per_row = (d_out + 3) >> 2;
    const int64_t idx = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
    if (idx >= static_cast<int64_t>(M) * per_row) return;
    const int tok = static_cast<int>(idx / per_row), o = static_cast<int>(idx - static_cast<int64_t>(tok) * per_row) * 4;
    const size_t plane = static_cast<size_t>(M) * d_out;
    const float *src = partial + static_cast<size_t>(tok) * d_out + o;
    unsigned short *dst = reinterpret_cast<unsigned short *>(y) + static_cast<size_t>(tok) * ldy + o;
    if (vec_ok) {
        float4 part[8];  // all loads first (splits <= 8), then the sum in split order
#pragma unroll
        for (int sp = 0; sp < 8; ++sp)
            part[sp] = sp < splits ? __ldcs(reinterpret_cast<const float4 *>(src + sp * plane)) : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 acc = part[0];
#pragma unroll
        for (int sp = 1; sp < 8; ++sp)
            if (sp < splits) acc.x += part[sp].x, acc.y += part[sp].y, acc.z += part[sp].z, acc.w += part[sp].w;
        uint2 out;
        out.x = Elem<BF16>::from_float(acc.x) | (static_cast<uint32_t>(Elem<BF16>::from_float(acc.y)) << 16);
        out.y = Elem<BF16>::from_float(acc.z) | (static_cast<uint32_t>(Elem<BF16>::from_float(acc.w)) << 16);
        *reinterpret_cast<uint2 *>(dst) = out;
    } else {
        for (int q = 0; q < 4 && o + q < d_out; ++q) {
            float acc = src[q];
            for (int sp = 1; sp < splits; ++sp) acc += src[sp * plane + q];
            dst[q] = Elem<BF16>::from_float(acc);
        }
    }
}

// ------------------------------------------------------------------ host side
}  // namespace

bool gemm_pair_enabled() { return true; }

namespace {
// fp16 row-major [rows, cols] with row pitch ld elements; box = 64 columns x box_rows rows, 128-byte swizzle
bool make_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    return make_map_2d(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, rows, cols, ld * 2, BK, box_rows,
                       CU_TENSOR_MAP_SWIZZLE_128B);
}

template <bool BF16, int AXIS, bool HAS_DELTA, bool GROUPED, int BN>
pd_status launch_one_t(const CUtensorMap &mw, const CUtensorMap &mx, const GemmArgs &args, int grid, cudaStream_t stream) {
    auto kernel = gemm_kernel<BF16, AXIS, HAS_DELTA, GROUPED, BN>;
    constexpr int smem = SmemLayout<BN>::kTotal;
    static std::atomic<bool> configured[kMaxDevices];  // per instantiation and device
    if (!ensure_dynamic_smem(kernel, smem, configured)) return PD_ERR_CUDA;
    kernel<<<grid, kNumThreads, smem, stream>>>(mw, mx, args);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace

namespace {

template <int AXIS, bool HAS_DELTA, bool GROUPED, int BN>
pd_status launch_one(const CUtensorMap &mw, const CUtensorMap &mx, const GemmArgs &args, int grid, cudaStream_t stream) {
    return args.bf16 ? launch_one_t<true, AXIS, HAS_DELTA, GROUPED, BN>(mw, mx, args, grid, stream)
                     : launch_one_t<false, AXIS, HAS_DELTA, GROUPED, BN>(mw, mx, args, grid, stream);
}

template <int BN>
pd_status launch_gemm_bn(const __half *x, int64_t M, int64_t ldx, const __half *w_b, const uint32_t *mask, const __half *v,
                         int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, uint32_t *status,
                         bool bf16, cudaStream_t stream) {
    CUtensorMap mw, mx;
    if (!make_map(&mw, w_b, d_out, d_in, d_in, BM) || !make_map(&mx, x, M, d_in, ldx, BN)) return PD_ERR_CUDA;
    GemmArgs args = {};
    args.mask = mask;
    args.v = v;
    args.y = y;
    args.ldy = ldy;
    args.M = static_cast<int>(M);
    args.d_out = static_cast<int>(d_out);
    args.d_in = static_cast<int>(d_in);
    args.tiles_m = static_cast<int>((d_out + BM - 1) / BM);
    args.tiles_n = static_cast<int>((M + BN - 1) / BN);
    args.k_steps = static_cast<int>((d_in + BK - 1) / BK);
    args.status = status;
    args.bf16 = bf16 ? 1 : 0;
    args.y_vec_ok = ((reinterpret_cast<uintptr_t>(y) & 15u) == 0 && ldy % 8 == 0) ? 1 : 0;
    const int tiles = args.tiles_m * args.tiles_n;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    if (mask == nullptr) return launch_one<PD_AXIS_ROW, false, false, BN>(mw, mx, args, grid, stream);
    if (axis == PD_AXIS_ROW) return launch_one<PD_AXIS_ROW, true, false, BN>(mw, mx, args, grid, stream);
    return launch_one<PD_AXIS_COL, true, false, BN>(mw, mx, args, grid, stream);
}

}  // namespace

namespace {

template <bool BF16, int AXIS, bool HAS_DELTA, bool GROUPED>
pd_status launch_pair_one_t(const CUtensorMap &mw, const CUtensorMap &mx, const GemmArgs &args, int grid, cudaStream_t stream) {
    auto kernel = gemm_pair_kernel<BF16, AXIS, HAS_DELTA, GROUPED>;
    constexpr int smem = PairLayout::kTotal;
    static std::atomic<bool> configured[kMaxDevices];  // per instantiation and device
    if (!ensure_dynamic_smem(kernel, smem, configured)) return PD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(pair_threads(GROUPED));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cuda_ok(cudaLaunchKernelEx(&cfg, kernel, mw, mx, args));
}

template <int AXIS, bool HAS_DELTA, bool GROUPED>
pd_status launch_pair_one(const CUtensorMap &mw, const CUtensorMap &mx, const GemmArgs &args, int grid, cudaStream_t stream) {
    return args.bf16 ? launch_pair_one_t<true, AXIS, HAS_DELTA, GROUPED>(mw, mx, args, grid, stream)
                     : launch_pair_one_t<false, AXIS, HAS_DELTA, GROUPED>(mw, mx, args, grid, stream);
}

// Tiles of 256 rows x 256 tokens on pairs of CTAs.
pd_status launch_gemm_pair(const __half *x, int64_t M, int64_t ldx, const __half *w_b, const uint32_t *mask, const __half *v,
                           int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, int token_tile, int splits,
                           float *partial, uint32_t *status, bool bf16, cudaStream_t stream) {
    CUtensorMap mw, mx;
    if (!make_map(&mw, w_b, d_out, d_in, d_in, BM) || !make_map(&mx, x, M, d_in, ldx, 128)) return PD_ERR_CUDA;
    GemmArgs args = {};
    args.mask = mask;
    args.v = v;
    args.y = y;
    args.ldy = ldy;
    args.M = static_cast<int>(M);
    args.d_out = static_cast<int>(d_out);
    args.d_in = static_cast<int>(d_in);
    args.tiles_m = static_cast<int>((d_out + BM - 1) / BM);
    args.tiles_n = static_cast<int>((M + token_tile - 1) / token_tile);
    args.token_tile = token_tile;
    args.k_steps = pair_split_steps(d_in, splits);  // per split; even: the MMA thread works on pairs of k steps
    args.splits = splits;
    args.partial = partial;
    args.status = status;
    args.bf16 = bf16 ? 1 : 0;
    args.y_vec_ok = ((reinterpret_cast<uintptr_t>(y) & 15u) == 0 && ldy % 8 == 0) ? 1 : 0;
    const int tiles = ((args.tiles_m + 1) / 2) * args.tiles_n * splits;
    const int pairs = tiles < sm_count() / 2 ? tiles : sm_count() / 2;
    pd_status st;
    if (mask == nullptr) st = launch_pair_one<PD_AXIS_ROW, false, false>(mw, mx, args, 2 * pairs, stream);
    else if (axis == PD_AXIS_ROW) st = launch_pair_one<PD_AXIS_ROW, true, false>(mw, mx, args, 2 * pairs, stream);
    else st = launch_pair_one<PD_AXIS_COL, true, false>(mw, mx, args, 2 * pairs, stream);
    if (st != PD_OK || splits == 1) return st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // scheduled while the GEMM runs; it waits on entry
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    const int64_t threads = M * ((d_out + 3) / 4);
    cfg.gridDim = dim3(static_cast<unsigned>((threads + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int vec_ok = (d_out % 4 == 0 && ldy % 4 == 0 && (reinterpret_cast<uintptr_t>(y) & 7u) == 0) ? 1 : 0;
    const int m32 = static_cast<int>(M), d32 = static_cast<int>(d_out);
    const float *cpartial = partial;
    count_launch();
    return cuda_ok(bf16 ? cudaLaunchKernelEx(&cfg, splitk_reduce_kernel<true>, cpartial, splits, m32, d32, y, ldy, vec_ok)
                        : cudaLaunchKernelEx(&cfg, splitk_reduce_kernel<false>, cpartial, splits, m32, d32, y, ldy, vec_ok));
}

// Multi-variant: token tiles of at most 256 sorted rows, one variant each.
pd_status launch_gemm_pair_grouped(const __half *x_sorted, int64_t M, const __half *w_b, const uint32_t *masks,
                                   int64_t mask_stride, const __half *vs, int64_t v_stride, unsigned long long col_axis_bits,
                                   int V, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, const int4 *tile_table,
                                   const int *n_token_tiles, int max_token_tiles, const int *row_index, uint32_t *status,
                                   bool bf16, cudaStream_t stream) {
    CUtensorMap mw, mx;
    if (!make_map(&mw, w_b, d_out, d_in, d_in, BM) || !make_map(&mx, x_sorted, M, d_in, d_in, 128)) return PD_ERR_CUDA;
    GemmArgs args = {};
    args.mask = masks;
    args.v = vs;
    args.y = y;
    args.ldy = ldy;
    args.M = static_cast<int>(M);
    args.d_out = static_cast<int>(d_out);
    args.d_in = static_cast<int>(d_in);
    args.tiles_m = static_cast<int>((d_out + BM - 1) / BM);
    args.tiles_n = 0;
    args.k_steps = static_cast<int>((d_in + 2 * BK - 1) / (2 * BK)) * 2;
    args.splits = 1;
    args.status = status;
    args.bf16 = bf16 ? 1 : 0;
    args.y_vec_ok = ((reinterpret_cast<uintptr_t>(y) & 15u) == 0 && ldy % 8 == 0) ? 1 : 0;
    args.tile_table = tile_table;
    args.n_token_tiles = n_token_tiles;
    args.row_index = row_index;
    args.mask_stride = mask_stride;
    args.v_stride = v_stride;
    args.col_axis_bits = col_axis_bits;
    args.V = V;
    const int64_t tiles = static_cast<int64_t>((args.tiles_m + 1) / 2) * max_token_tiles;  // upper bound; the kernel reads the real count
    const int pairs = tiles < sm_count() / 2 ? static_cast<int>(tiles) : sm_count() / 2;
    return launch_pair_one<PD_AXIS_ROW, true, true>(mw, mx, args, 2 * pairs, stream);
}

}  // namespace

namespace {

// Token tile and number of k splits of the pair kernel.  Measured: a pair of k steps costs at least about 1250 clocks
// whatever the tile's width, and 4 clocks per token plus 400 when that is more; a tile costs about 3000 clocks to
// start and drain.  With few tokens the tiles are too few for the 74 CTA pairs: the k steps are then
// dealt to several tiles whose fp32 partial sums a second kernel adds (about 5000 clocks plus its traffic).  Picks
// the cheapest estimate; ties go to fewer splits, then to the narrower tile (more CTAs stream the weights).
void pair_plan(int64_t M, int64_t d_out, int64_t d_in, int sms, int *token_tile, int *splits) {
    const int64_t tiles_m2 = (d_out + 2 * BM - 1) / (2 * BM);
    const int pairs = sms / 2 > 0 ? sms / 2 : 1;
    const int64_t k_pairs = (d_in + 2 * BK - 1) / (2 * BK);
    int64_t best_cost = -1;
    for (int sp = 1; sp <= 8; ++sp) {
        if (sp > 1 && (M > 1024 || k_pairs / sp < 4)) break;
        for (int tt = 256; tt >= 64; tt >>= 1) {
            const int64_t units = tiles_m2 * ((M + tt - 1) / tt) * sp;
            const int64_t per_pair = 4 * tt + 400 > 1250 ? 4 * tt + 400 : 1250;
            const int64_t per_unit = ((k_pairs + sp - 1) / sp) * per_pair + 3000;
            int64_t cost = ((units + pairs - 1) / pairs) * per_unit;
            if (sp > 1) cost += 5000 + (M * d_out * (sp + 1)) / 2048;  // the reduction: ~4 bytes per partial at ~2 KB per clock
            if (best_cost < 0 || cost < best_cost || (cost == best_cost && sp == *splits)) *token_tile = tt, *splits = sp, best_cost = cost;
        }
    }
}

}  // namespace

int pair_split_steps(int64_t d_in, int splits) {
    const int64_t k_pairs = (d_in + 2 * BK - 1) / (2 * BK);
    return static_cast<int>((k_pairs + splits - 1) / splits) * 2;
}

size_t gemm_partial_bytes(int64_t M, int64_t d_out, int64_t d_in) {
    if (!(gemm_pair_enabled() && d_out >= 256)) return 0;
    int tt = 256, splits = 1;
    pair_plan(M, d_out, d_in, sm_count(), &tt, &splits);
    return splits > 1 ? round_up(static_cast<size_t>(splits) * M * d_out * 4, 256) : 0;
}

pd_status launch_gemm(const __half *x, int64_t M, int64_t ldx, const __half *w_b, const uint32_t *mask,
                      const __half *v, int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy,
                      float *partial, uint32_t *status, bool bf16, cudaStream_t stream) {
    const int sms = sm_count();
    if (gemm_pair_enabled() && d_out >= 256) {
        // CTA pairs, tiles of 256 rows x token_tile tokens, the k loop split when the tiles are too few (pair_plan).
        int tt = 256, splits = 1;
        pair_plan(M, d_out, d_in, sms, &tt, &splits);
        if (splits > 1 && partial == nullptr) return PD_ERR_WORKSPACE;
        return launch_gemm_pair(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, tt, splits, partial, status, bf16, stream);
    }
    // One CTA per tile (fewer than 256 output rows).  256 tokens per tile amortise the W_hat transform best, but with
    // few tokens that leaves most SMs without
    // a tile (M = 256 on a 4096-row layer: 32 tiles).  Estimated time = waves x per-stage time, where a stage
    // costs the MMA (2 clocks per token) but never less than the transform/handshake floor; ties go to the
    // smaller tile, which spreads the weight stream over more SMs.
    const int64_t tiles_m = (d_out + BM - 1) / BM;
    int best = 256;
    int64_t best_cost = -1;
    for (int bn = 256; bn >= 64; bn >>= 1) {
        const int64_t tiles = tiles_m * ((M + bn - 1) / bn);
        const int64_t cost = ((tiles + sms - 1) / sms) * (2 * bn > 400 ? 2 * bn : 400);
        if (best_cost < 0 || cost <= best_cost) best = bn, best_cost = cost;
    }
    if (best == 256) return launch_gemm_bn<256>(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, status, bf16, stream);
    if (best == 128) return launch_gemm_bn<128>(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, status, bf16, stream);
    return launch_gemm_bn<64>(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, status, bf16, stream);
}

namespace {

template <int BN>
pd_status launch_gemm_grouped_bn(const __half *x_sorted, int64_t M, const __half *w_b, const uint32_t *masks,
                              int64_t mask_stride, const __half *vs, int64_t v_stride, unsigned long long col_axis_bits,
                              int V, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, const int4 *tile_table,
                              const int *n_token_tiles, int max_token_tiles, const int *row_index, uint32_t *status,
                              bool bf16, cudaStream_t stream) {
    CUtensorMap mw, mx;
    if (!make_map(&mw, w_b, d_out, d_in, d_in, BM) || !make_map(&mx, x_sorted, M, d_in, d_in, BN)) return PD_ERR_CUDA;
    GemmArgs args = {};
    args.mask = masks;
    args.v = vs;
    args.y = y;
    args.ldy = ldy;
    args.M = static_cast<int>(M);
    args.d_out = static_cast<int>(d_out);
    args.d_in = static_cast<int>(d_in);
    args.tiles_m = static_cast<int>((d_out + BM - 1) / BM);
    args.tiles_n = 0;
    args.k_steps = static_cast<int>((d_in + BK - 1) / BK);
    args.status = status;
    args.bf16 = bf16 ? 1 : 0;
    args.y_vec_ok = ((reinterpret_cast<uintptr_t>(y) & 15u) == 0 && ldy % 8 == 0) ? 1 : 0;
    args.tile_table = tile_table;
    args.n_token_tiles = n_token_tiles;
    args.row_index = row_index;
    args.mask_stride = mask_stride;
    args.v_stride = v_stride;
    args.col_axis_bits = col_axis_bits;
    args.V = V;
    const int64_t tiles = static_cast<int64_t>(args.tiles_m) * max_token_tiles;  // upper bound; the kernel reads the real count
    const int grid = tiles < sm_count() ? static_cast<int>(tiles) : sm_count();
    return launch_one<PD_AXIS_ROW, true, true, BN>(mw, mx, args, grid, stream);
}

}  // namespace

pd_status launch_gemm_grouped(const __half *x_sorted, int64_t M, const __half *w_b, const uint32_t *masks,
                              int64_t mask_stride, const __half *vs, int64_t v_stride, unsigned long long col_axis_bits,
                              int V, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, const int4 *tile_table,
                              const int *n_token_tiles, int max_token_tiles, int token_tile, const int *row_index,
                              uint32_t *status, bool bf16, cudaStream_t stream) {
    if (token_tile == 256 && gemm_pair_enabled() && d_out >= 256)
        return launch_gemm_pair_grouped(x_sorted, M, w_b, masks, mask_stride, vs, v_stride, col_axis_bits, V, d_out, d_in, y, ldy,
                                        tile_table, n_token_tiles, max_token_tiles, row_index, status, bf16, stream);
#define PD_GROUPED(BN)                                                                                                     \
    return launch_gemm_grouped_bn<BN>(x_sorted, M, w_b, masks, mask_stride, vs, v_stride, col_axis_bits, V, d_out, d_in, y, \
                                      ldy, tile_table, n_token_tiles, max_token_tiles, row_index, status, bf16, stream)
    if (token_tile == 64) PD_GROUPED(64);
    if (token_tile == 128) PD_GROUPED(128);
    PD_GROUPED(256);
#undef PD_GROUPED
}

}  // namespace pd
