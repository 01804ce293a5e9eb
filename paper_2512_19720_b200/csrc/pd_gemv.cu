// Decode path: y[M<=16, d_out] = x . (W_b + v (.) B)^T, bound by HBM (2.125 bytes per weight element).
//
// gemv_stream_kernel (below) is the product path for every d_in that is a multiple of 128; gemv_generic_kernel
// (one warp per output row, plain FMAs) covers the remaining shapes and is not tuned.
#include "pd_ptx.cuh"

namespace pd {
namespace {

// arguments of the generic kernel
struct GemvArgs {
    const __half *x;
    const __half *w_b;
    const uint32_t *mask;  // nullptr: base only
    const __half *v;
    __half *y;
    int64_t ldx, ldy;
    int M, d_out, d_in;
    // grouped mode (multi-variant): the tokens of this launch are rows
    // row_index[group_offsets[group] .. group_offsets[group + 1]) of x and y; M is ignored
    const int *row_index;
    const int *group_offsets;
    int group;
};

// ---------------------------------------------------------------------------------------------
// Streaming decode kernel: weights brought in by TMA, one CTA per 16 output rows, two or three CTAs per SM.
//
// A CTA owns 16 rows for the whole of d_in, so its result needs no other CTA: no partial sums in
// global memory, no tickets, no fences.  It walks d_in in steps of 512 columns: 1 KB of contiguous
// W_b per row and step (HBM wants long row segments: on B200 a pure TMA stream of [16 rows x 2 KB]
// steps measured 6.1-7.1 TB/s on the 7B shapes against 4.4-5.4 TB/s for 512-byte segments; 1 KB
// steps run as fast as 2 KB ones here and halve what the consumers still have to do once the last
// bytes have landed).  A step is 16 KB of W_b in two boxes of {64 columns, 4 blocks, 16 rows}
// (128-byte swizzle; rows of 512 bytes keep the fragment reads conflict free), one box of mask
// words and, for the col axis, a bulk copy of the step's scales: 17-18 KB.  A CTA keeps six steps
// in flight (two CTAs per SM), or four (three CTAs per SM) when the grid is large enough.
//
// The mask box is fetched through a map that sees the words as {4 words, rows, groups of 128
// columns}: in shared memory the 16 bytes of one row and group sit next to those of the next row,
// so the eight rows a warp reads at once fall into different banks.
//
// Eight consumer warps share every step: each takes one 64-column block and all 16 rows.  W_b, mask
// and the col-axis scales come from shared memory; the x fragments are read straight from global
// memory -- x is small and L2-resident, and keeping it out of shared memory leaves the ring to the
// weights.  With more than 8 tokens the token index is the MMA's M (16) and 8 rows its N; with up to 8
// tokens the 16 rows are M and the tokens N, which halves the number of MMAs.  W_hat = W_b +- s with
// s = v[row] (row axis) or s = v[k] (col axis) is formed in fp16 registers (add.f16x2: one rounding,
// as the merge and the prefill path form it) and multiplied with fp32 accumulation.  The eight warps' partial
// sums are added in warp order through shared memory.
//
// Programmatic dependent launch: the kernel may start while the previous kernel in the stream drains.  The
// consumers wait for that kernel (griddepcontrol.wait) before they touch x or y; the producer waits too, unless
// the caller has declared the weights resident (PD_LINEAR_WEIGHTS_RESIDENT), in which case it streams W_b, mask
// and v at once.
constexpr int kStreamConsumers = 8;
constexpr int kStreamThreads = (kStreamConsumers + 1) * 32;
constexpr int kStreamRows = 16;             // output rows per CTA
// one stage of KS columns: W_b boxes of [16 rows][4 blocks][128 B], swizzled; mask as [groups of 128 columns]
// [rows][4 words]; the step's col-axis scales.  36 bytes per column: every stage starts 1024-byte aligned.
constexpr int kStW = 0;
__host__ __device__ constexpr int stage_mask_offset(int ks) { return kStreamRows * ks * 2; }
__host__ __device__ constexpr int stage_v_offset(int ks) { return stage_mask_offset(ks) + kStreamRows * ks / 8; }
__host__ __device__ constexpr int stage_bytes(int ks) { return stage_v_offset(ks) + ks * 2; }
constexpr int kRedOffset = 0;               // [8 warps][16 tokens][R rows] fp32, over the ring once it has drained
static_assert(kStreamConsumers * 16 * kStreamRows * 4 <= stage_bytes(512), "the reduction buffer reuses stage 0");
static_assert(stage_bytes(512) % 1024 == 0 && stage_bytes(1024) % 1024 == 0, "stage alignment");
constexpr int stream_smem_bytes(int ks, int stages) { return stages * stage_bytes(ks) + 256 + 1024 /* alignment slack */; }
// three CTAs per SM when a CTA's ring is at most 72 KB (and the registers are capped accordingly)
__host__ __device__ constexpr bool stream_three_per_sm(int ks, int stages) { return stages * stage_bytes(ks) <= 72 * 1024; }

struct StreamArgs {
    const __half *x;
    const __half *v;
    __half *y;
    int64_t ldx, ldy;
    int M, d_out, d_in;
    int n_k;      // steps of KS columns (the last one may be partly past d_in)
    int weights_resident;  // W_b, mask and v are not written by earlier work on the stream: load them before the grid dependency resolves
    uint32_t *status;
};

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint4 ldg_cached(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// x fragments of one 64-column block: [c] = piece t + 4c; a = token g, b = token g + 8
struct XFrag {
    uint4 a[2], b[2];
};

template <bool COL, bool M16>
__device__ __forceinline__ void load_xfrag(XFrag &f, const StreamArgs &a, int k0, int g, int t) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const int k = k0 + 8 * (t + 4 * c);
        f.a[c] = make_uint4(0, 0, 0, 0);
        f.b[c] = make_uint4(0, 0, 0, 0);
        if (g < a.M) f.a[c] = ldg_cached(a.x + static_cast<size_t>(g) * a.ldx + k);
        if (M16 && g + 8 < a.M) f.b[c] = ldg_cached(a.x + static_cast<size_t>(g + 8) * a.ldx + k);
    }
}

template <bool BF16, int AXIS, bool HAS_DELTA, bool M16, int KS, int STAGES>
__global__ void __maxnreg__(stream_three_per_sm(KS, STAGES) ? 72 : 96)
gemv_stream_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_m, const StreamArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float *red = reinterpret_cast<float *>(smem + kRedOffset);
    constexpr int kStreamStages = STAGES;
    constexpr int R = kStreamRows;
    constexpr int kStageBytes = stage_bytes(KS), kStMask = stage_mask_offset(KS), kStV = stage_v_offset(KS);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + STAGES * kStageBytes);
    uint64_t *empty = full + kStreamStages;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(empty + kStreamStages);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool kCol = HAS_DELTA && AXIS == PD_AXIS_COL;
    constexpr uint32_t kTxBytes = static_cast<uint32_t>(kStreamRows) * (KS * 2u + (HAS_DELTA ? KS / 8u : 0u));
    constexpr int kStep = KS;                  // columns per step
    constexpr int kItems = kStep / 64 / kStreamConsumers;  // 64-column blocks per warp and step
    constexpr int kTiles = R / 8;              // n8 tiles of output rows
    static_assert(KS == 512 || KS == 1024, "columns per step");

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStreamStages; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, kStreamConsumers);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == kStreamConsumers) {
        // ------------------------------------------------ producer
        if (lane == 0) {
            grid_launch_dependents();  // the next kernel in the stream may start its own weight loads
            // Unless the caller vouches that no earlier work on the stream writes the weights, they may be the
            // previous kernel's output (pd_pack_delta or pd_merge right before this call): wait for it like the consumers.
            if (!a.weights_resident) grid_dependency_wait();
            uint32_t gs = 0;           // steps issued so far
            bool ok = true;
            {
                const int row0 = blockIdx.x * R;
                for (int s = 0; s < a.n_k; ++s, ++gs) {
                    const int st = gs % kStreamStages;
                    if (gs >= kStreamStages &&
                        !(ok = mbar_wait(empty + st, ((gs / kStreamStages) & 1) ^ 1, abort_flag, a.status, 11)))
                        break;
                    unsigned char *base = smem + st * kStageBytes;
                    const uint32_t v_bytes = kCol ? static_cast<uint32_t>(min(kStep, a.d_in - s * kStep) * 2) : 0u;
                    mbar_arrive_expect_tx(full + st, kTxBytes + v_bytes);
#pragma unroll
                    for (int q = 0; q < kStep / 256; ++q)
                        tma_load_3d(&map_w, full + st, base + kStW + q * (R * 512), 0, s * (kStep / 64) + 4 * q, row0);
                    if (HAS_DELTA) tma_load_3d(&map_m, full + st, base + kStMask, 0, row0, s * (kStep / 128));
                    if (kCol) bulk_load_1d(base + kStV, a.v + static_cast<size_t>(s) * kStep, v_bytes, full + st);
                }
            }
        }
    } else {
        // ------------------------------------------------ consumers
        const int g = lane >> 2, t = lane & 3;
        const uint32_t byte_t = static_cast<uint32_t>(t) | 0x4440u;  // prmt: byte t of the first operand, zeros above
        grid_dependency_wait();  // x may be the previous kernel's output
        const int n_items = kItems * a.n_k;
        auto item_k0 = [&](int it) { return (it / kItems) * kStep + (kItems * warp + (it % kItems)) * 64; };
        uint32_t gs = 0;  // steps consumed so far
        bool ok = true;
        const int row0 = blockIdx.x * R;
        float acc[kTiles][4];
#pragma unroll
        for (int j = 0; j < kTiles; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
        uint32_t mag[kTiles];  // |B operand| of the delta MMA as a half2: (s, s) for the row axis, (1, 1) for the col axis
#pragma unroll
        for (int j = 0; j < kTiles; ++j) {
            mag[j] = Elem<BF16>::kOnePair;
            if (HAS_DELTA && AXIS == PD_AXIS_ROW)
                mag[j] = Elem<BF16>::scale_pair(*reinterpret_cast<const unsigned short *>(a.v + min(row0 + 8 * j + g, a.d_out - 1)));
        }
        // items: (step s, block bb of this warp), k0 = s*kStep + (kItems*warp + bb)*64; x fragments one item ahead
        // (two ahead for up to 8 tokens, where the registers allow it: the loads come from L2, ~1 us away under load)
        constexpr int kAhead = M16 ? 1 : 2;
        XFrag cur, nxt, nxt2;
        if (item_k0(0) < a.d_in) load_xfrag<kCol, M16>(cur, a, item_k0(0), g, t);
        if (kAhead == 2 && 1 < n_items && item_k0(1) < a.d_in) load_xfrag<kCol, M16>(nxt, a, item_k0(1), g, t);
        for (int it = 0; it < n_items && ok; ++it) {
            const int bb = it % kItems, st = gs % kStreamStages;
            const int k0 = item_k0(it);
            if (kAhead == 1) {
                if (it + 1 < n_items && item_k0(it + 1) < a.d_in) load_xfrag<kCol, M16>(nxt, a, item_k0(it + 1), g, t);
            } else {
                if (it + 2 < n_items && item_k0(it + 2) < a.d_in) load_xfrag<kCol, M16>(nxt2, a, item_k0(it + 2), g, t);
            }
            if (bb == 0 && !(ok = mbar_wait(full + st, (gs / kStreamStages) & 1, abort_flag, a.status, 12))) break;
            if (k0 < a.d_in) {  // else past the end of d_in: W was zero-filled there and x must not be read
                const int blk = kItems * warp + bb;                   // block inside the step
                const unsigned char *stage = smem + st * kStageBytes;
                const unsigned char *box = stage + kStW + (blk >> 2) * (R * 512);
                const int bi = blk & 3;                               // block inside its box
                uint2 mw[kTiles];                                     // the block's 64 sign bits of rows 8j + g
                if (HAS_DELTA) {
#pragma unroll
                    for (int j = 0; j < kTiles; ++j)
                        mw[j] = *reinterpret_cast<const uint2 *>(stage + kStMask + (blk >> 1) * (R * 16) + (8 * j + g) * 16 + (blk & 1) * 8);
                }
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    // byte offset inside a 512-byte row of the box, swizzled: piece index ^ (bits 7..9 of the offset)
                    const uint32_t in_row = static_cast<uint32_t>(bi * 128) +
                                            ((static_cast<uint32_t>(t + 4 * c) ^ static_cast<uint32_t>(((g & 1) << 2) | bi)) << 4);
                    const uint4 xa = cur.a[c], xb = cur.b[c];
                    // |B operand| of the delta MMA for the four half2 pairs of this piece: v[k] itself (col axis),
                    // read from the stage (all lanes with the same t read the same 16 bytes: a broadcast)
                    uint4 vv = make_uint4(0, 0, 0, 0);
                    if (kCol) {
                        vv = *reinterpret_cast<const uint4 *>(stage + kStV + (blk * 64 + 8 * (t + 4 * c)) * 2);
                        if (BF16) {  // the scales arrive as binary16: one rounding to the weights' type
                            vv.x = Elem<BF16>::scale_pair2(vv.x), vv.y = Elem<BF16>::scale_pair2(vv.y);
                            vv.z = Elem<BF16>::scale_pair2(vv.z), vv.w = Elem<BF16>::scale_pair2(vv.w);
                        }
                    }
                    if (M16) {
    #pragma unroll
                        for (int j = 0; j < kTiles; ++j) {
                            uint4 w = *reinterpret_cast<const uint4 *>(box + (8 * j + g) * 512 + in_row);
                            if (HAS_DELTA) {
                                // the piece's 8 sign bits are byte t of word c.  b * 0x8001 puts bit i at i and i + 15,
                                // so a left shift by 15 - 2r brings bit 2r to bit 15 and bit 2r + 1 to bit 31: the signs
                                // of halves 2r, 2r + 1.  A clear bit (B = -1) flips the sign of the magnitude.
                                const uint32_t sp = prmt(c ? mw[j].y : mw[j].x, 0u, byte_t) * 0x8001u;
                                const uint32_t pm0 = lop3_andn_xor(sp << 15, 0x80008000u, kCol ? vv.x : mag[j]);
                                const uint32_t pm1 = lop3_andn_xor(sp << 13, 0x80008000u, kCol ? vv.y : mag[j]);
                                const uint32_t pm2 = lop3_andn_xor(sp << 11, 0x80008000u, kCol ? vv.z : mag[j]);
                                const uint32_t pm3 = lop3_andn_xor(sp << 9, 0x80008000u, kCol ? vv.w : mag[j]);
                                // W_hat = W_b +- v in the weights' 16-bit type, as the merge and the prefill path form it: one MMA per
                                // 16 columns instead of one for W_b and one for the signs
                                w.x = Elem<BF16>::add2(w.x, pm0), w.y = Elem<BF16>::add2(w.y, pm1);
                                w.z = Elem<BF16>::add2(w.z, pm2), w.w = Elem<BF16>::add2(w.w, pm3);
                            }
                            Elem<BF16>::mma16816(acc[j], xa.x, xb.x, xa.y, xb.y, w.x, w.y);
                            Elem<BF16>::mma16816(acc[j], xa.z, xb.z, xa.w, xb.w, w.z, w.w);
                        }
                    } else {
                        // up to 8 tokens: the 16 rows are the MMA's M and the tokens its N, so one MMA does what two
                        // do above (A = the W_b pieces of rows g and g + 8, B = token g's piece of x);
                        // acc[c] = {row g: tokens 2t, 2t+1; row g + 8: tokens 2t, 2t+1}
                        uint4 w0 = *reinterpret_cast<const uint4 *>(box + g * 512 + in_row);
                        uint4 w1 = *reinterpret_cast<const uint4 *>(box + (8 + g) * 512 + in_row);
                        if (HAS_DELTA) {
                            uint32_t pm[2][4];
#pragma unroll
                            for (int j = 0; j < 2; ++j) {  // sign expansion as above
                                const uint32_t sp = prmt(c ? mw[j].y : mw[j].x, 0u, byte_t) * 0x8001u;
                                pm[j][0] = lop3_andn_xor(sp << 15, 0x80008000u, kCol ? vv.x : mag[j]);
                                pm[j][1] = lop3_andn_xor(sp << 13, 0x80008000u, kCol ? vv.y : mag[j]);
                                pm[j][2] = lop3_andn_xor(sp << 11, 0x80008000u, kCol ? vv.z : mag[j]);
                                pm[j][3] = lop3_andn_xor(sp << 9, 0x80008000u, kCol ? vv.w : mag[j]);
                            }
                            w0.x = Elem<BF16>::add2(w0.x, pm[0][0]), w0.y = Elem<BF16>::add2(w0.y, pm[0][1]);
                            w0.z = Elem<BF16>::add2(w0.z, pm[0][2]), w0.w = Elem<BF16>::add2(w0.w, pm[0][3]);
                            w1.x = Elem<BF16>::add2(w1.x, pm[1][0]), w1.y = Elem<BF16>::add2(w1.y, pm[1][1]);
                            w1.z = Elem<BF16>::add2(w1.z, pm[1][2]), w1.w = Elem<BF16>::add2(w1.w, pm[1][3]);
                        }
                        // the two pieces of a block go to accumulators of their own: two short chains of dependent MMAs
                        Elem<BF16>::mma16816(acc[c], w0.x, w1.x, w0.y, w1.y, xa.x, xa.y);
                        Elem<BF16>::mma16816(acc[c], w0.z, w1.z, w0.w, w1.w, xa.z, xa.w);
                    }
                }
            }
            if (bb == kItems - 1) {
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + st);
                ++gs;
            }
            cur = nxt;
            if (kAhead == 2) nxt = nxt2;
        }

        // ---- add the eight warps' partial sums in warp order.  The first barrier ORs "a wait ran out"
        // over the consumers, so that all of them leave together.
        uint32_t gave_up;
        asm volatile(
            "{\n"
            ".reg .pred p, q;\n"
            "setp.ne.u32 q, %1, 0;\n"
            "bar.red.or.pred p, 1, %2, q;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(gave_up)
            : "r"(static_cast<uint32_t>(!ok || *abort_flag)), "n"(kStreamConsumers * 32)
            : "memory");
        if (!gave_up) {
            float *mine = red + warp * 16 * R;  // [16 tokens][R rows]
            if (M16) {
#pragma unroll
                for (int j = 0; j < kTiles; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int ol = 8 * j + 2 * t + e;
                        mine[g * R + ol] = acc[j][e];
                        mine[(g + 8) * R + ol] = acc[j][2 + e];
                    }
            } else {  // tokens 2t, 2t + 1 of rows g and g + 8
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    mine[(2 * t + e) * R + g] = acc[0][e] + acc[1][e];
                    mine[(2 * t + e) * R + g + 8] = acc[0][2 + e] + acc[1][2 + e];
                }
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kStreamConsumers * 32) : "memory");
            for (int idx = threadIdx.x; idx < (M16 ? 16 : 8) * R; idx += kStreamConsumers * 32) {  // (token, row) pairs
                const int tok = idx / R, ol = idx % R;
                float sum = 0.f;
#pragma unroll
                for (int w = 0; w < kStreamConsumers; ++w) sum += red[(w * 16 + tok) * R + ol];
                if (tok < a.M && row0 + ol < a.d_out)
                    reinterpret_cast<unsigned short *>(a.y)[static_cast<size_t>(tok) * a.ldy + row0 + ol] = Elem<BF16>::from_float(sum);
            }
        }
    }
}

// Any d_in that is a multiple of 32 (the tensor path above needs a multiple of 128): one warp per
// output row, plain fp32 FMAs, shuffle reduction.  Correctness path for odd shapes, not tuned.
template <bool BF16, int AXIS>
__global__ void __launch_bounds__(256) gemv_generic_kernel(const GemvArgs a) {
    const unsigned short *w_bits = reinterpret_cast<const unsigned short *>(a.w_b), *x_bits = reinterpret_cast<const unsigned short *>(a.x);
    const int lane = threadIdx.x & 31;
    const int o = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (o >= a.d_out) return;
    int n_tok = a.M;
    const int *tok_rows = nullptr;
    if (a.group_offsets != nullptr) {
        const int first = a.group_offsets[a.group];
        n_tok = a.group_offsets[a.group + 1] - first;
        tok_rows = a.row_index + first;
    }
  for (int tok0 = 0; tok0 < n_tok; tok0 += 16) {
    const int M = min(16, n_tok - tok0);
    float base[16], delta[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) base[m] = delta[m] = 0.f;
    const int words = a.d_in >> 5;
    for (int w = lane; w < words; w += 32) {
        const uint32_t word = a.mask ? a.mask[static_cast<size_t>(o) * words + w] : 0u;
        for (int b = 0; b < 32; ++b) {
            const int k = 32 * w + b;
            const float wv = Elem<BF16>::to_float(w_bits[static_cast<size_t>(o) * a.d_in + k]);
            float sg = ((word >> b) & 1u) ? 1.f : -1.f;
            if (AXIS == PD_AXIS_COL && a.mask) sg *= __half2float(a.v[k]);
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                if (m < M) {
                    const int xr = tok_rows ? tok_rows[tok0 + m] : tok0 + m;
                    const float xv = Elem<BF16>::to_float(x_bits[static_cast<size_t>(xr) * a.ldx + k]);
                    base[m] = fmaf(xv, wv, base[m]);
                    delta[m] = fmaf(xv, sg, delta[m]);
                }
            }
        }
    }
    const float s = !a.mask ? 0.f : (AXIS == PD_AXIS_ROW ? __half2float(a.v[o]) : 1.f);
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        if (m < M) {
            float val = base[m] + s * delta[m];
#pragma unroll
            for (int sft = 16; sft > 0; sft >>= 1) val += __shfl_xor_sync(0xffffffffu, val, sft);
            const int yr = tok_rows ? tok_rows[tok0 + m] : tok0 + m;
            if (lane == 0) reinterpret_cast<unsigned short *>(a.y)[static_cast<size_t>(yr) * a.ldy + o] = Elem<BF16>::from_float(val);
        }
    }
  }
}

template <bool BF16, int AXIS, bool HAS_DELTA, bool M16, int KS, int STAGES>
pd_status launch_stream_variant(const CUtensorMap &mw, const CUtensorMap &mm, const StreamArgs &args, int grid,
                                cudaStream_t stream) {
    auto kernel = gemv_stream_kernel<BF16, AXIS, HAS_DELTA, M16, KS, STAGES>;
    constexpr int kStreamSmem = stream_smem_bytes(KS, STAGES);
    static std::atomic<bool> configured[kMaxDevices];  // per instantiation and device
    if (!ensure_dynamic_smem(kernel, kStreamSmem, configured)) return PD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = kStreamSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may start while the previous kernel drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cuda_ok(cudaLaunchKernelEx(&cfg, kernel, mw, mm, args));
}

template <int KS, int STAGES>
pd_status launch_stream_rows(const __half *x, int M, int64_t ldx, const __half *w_b, const uint32_t *mask, const __half *v,
                             int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, uint32_t *status,
                             bool weights_resident, bool bf16, cudaStream_t stream) {
    constexpr int step = KS, R = kStreamRows;
    const bool m16 = M > 8, delta = mask != nullptr;
    CUtensorMap mw, mm;
    if (!make_map_blocked_f16(&mw, w_b, d_out, d_in, d_in * 2, 4, R)) return PD_ERR_CUDA;
    mm = mw;
    if (delta && !make_map_mask_groups(&mm, mask, d_out, d_in, R, step / 128)) return PD_ERR_CUDA;
    StreamArgs a;
    a.x = x;
    a.v = v;
    a.y = y;
    a.ldx = ldx;
    a.ldy = ldy;
    a.M = M;
    a.d_out = static_cast<int>(d_out);
    a.d_in = static_cast<int>(d_in);
    a.n_k = static_cast<int>((d_in + step - 1) / step);
    a.weights_resident = weights_resident ? 1 : 0;
    a.status = status;
    // one CTA per tile of R rows: a persistent grid walking several tiles measured slower on the 7B
    // shapes (fewer rings in flight, more registers)
    const int grid = static_cast<int>((d_out + R - 1) / R);
#define PD_STREAM_CASE(AX, D, W)                                                                      \
    return bf16 ? launch_stream_variant<true, AX, D, W, KS, STAGES>(mw, mm, a, grid, stream)          \
                : launch_stream_variant<false, AX, D, W, KS, STAGES>(mw, mm, a, grid, stream)
    if (!delta) {
        if (m16) PD_STREAM_CASE(PD_AXIS_ROW, false, true);
        PD_STREAM_CASE(PD_AXIS_ROW, false, false);
    }
    if (axis == PD_AXIS_ROW) {
        if (m16) PD_STREAM_CASE(PD_AXIS_ROW, true, true);
        PD_STREAM_CASE(PD_AXIS_ROW, true, false);
    }
    if (m16) PD_STREAM_CASE(PD_AXIS_COL, true, true);
    PD_STREAM_CASE(PD_AXIS_COL, true, false);
#undef PD_STREAM_CASE
}

pd_status launch_stream(const __half *x, int M, int64_t ldx, const __half *w_b, const uint32_t *mask, const __half *v,
                        int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy, uint32_t *status,
                        bool weights_resident, bool bf16, cudaStream_t stream) {
    // Ring depth.  A shorter ring (four steps, 72 KB) lets three CTAs share an SM: the same bytes in flight,
    // but a CTA that is finishing (last step, reduction, store) overlaps two that stream.  It needs a grid that
    // fills three CTAs per SM (smaller grids need six steps per CTA to keep enough in flight) and whose last
    // wave is not much emptier than with two CTAs per SM.  Measured and dropped: tiles of 32 rows (half the x
    // traffic, but too few consumer warps per SM on small grids) and tiles of 12-15 rows (fill every SM when
    // d_out / 16 is just under a wave, but the consumers' work per CTA does not shrink with the tile).
    const double tiles = static_cast<double>((d_out + kStreamRows - 1) / kStreamRows);
    const double w3 = tiles / (3.0 * sm_count()), w2 = tiles / (2.0 * sm_count());
    const bool three = w3 >= 1.0 && w3 / ceil(w3) >= w2 / ceil(w2) - 0.1;
    if (three) return launch_stream_rows<512, 4>(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, status, weights_resident, bf16, stream);
    return launch_stream_rows<512, 6>(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, status, weights_resident, bf16, stream);
}

}  // namespace

pd_status launch_gemv(const __half *x, int M, int64_t ldx, const __half *w_b, const uint32_t *mask,
                      const __half *v, int axis, int64_t d_out, int64_t d_in, __half *y, int64_t ldy,
                      const int *row_index, const int *group_offsets, int group, const GemvScratch *ws,
                      cudaStream_t stream) {
    // plain calls on TMA-friendly shapes stream the weights through shared memory
    if (ws != nullptr && group_offsets == nullptr && d_in % 128 == 0)
        return launch_stream(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, ws->status, ws->weights_resident, ws->bf16, stream);
    GemvArgs args;
    args.x = x;
    args.w_b = w_b;
    args.mask = mask;
    args.v = v;
    args.y = y;
    args.ldx = ldx;
    args.ldy = ldy;
    args.M = M;
    args.d_out = static_cast<int>(d_out);
    args.d_in = static_cast<int>(d_in);
    args.row_index = row_index;
    args.group_offsets = group_offsets;
    args.group = group;
    const int rows_per_cta = 8;
    const unsigned grid = static_cast<unsigned>((d_out + rows_per_cta - 1) / rows_per_cta);
    const bool bf16 = ws != nullptr && ws->bf16;
    if (axis == PD_AXIS_ROW) {
        if (bf16) gemv_generic_kernel<true, PD_AXIS_ROW><<<grid, 256, 0, stream>>>(args);
        else gemv_generic_kernel<false, PD_AXIS_ROW><<<grid, 256, 0, stream>>>(args);
    } else {
        if (bf16) gemv_generic_kernel<true, PD_AXIS_COL><<<grid, 256, 0, stream>>>(args);
        else gemv_generic_kernel<false, PD_AXIS_COL><<<grid, 256, 0, stream>>>(args);
    }
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace pd
