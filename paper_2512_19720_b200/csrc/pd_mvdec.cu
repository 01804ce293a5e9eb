// Multi-variant decode: y[m, :] = x[m, :] . (W_b + v_g (.) B_g)^T with g = ids[m], for a batch of up to 64 token
// rows that carry their own variant id, in ONE pass over W_b.  HBM traffic: 2 bytes of W_b per weight element plus
// 1/8 byte of mask per element and variant present in the batch.
//
// Decomposition
//   - A CTA owns 64 output rows and one slice of d_in; the CTAs of a cluster (1..8) own consecutive slices of the
//     same rows and add their partial sums through distributed shared memory in rank order, so the result does
//     not depend on scheduling.
//   - Every CTA buckets the (at most 64) token rows by variant id itself -- a few hundred comparisons, cheaper than
//     a separate launch -- and cuts each variant's rows into "items" of at most 8 tokens: one item is one n8 tile
//     of a warp-level m16n8k16 MMA whose M dimension is 16 output rows.  An item costs two MMAs per 16 columns:
//     A = W_b fragment (shared by all items) and A = +-v fragment built from the item's own mask words, both
//     against the same x fragment and into the same fp32 accumulator.
//   - Steps of 128 columns flow through a 3-stage ring: a producer lane issues TMA loads of the W_b tile
//     (two 128-byte-swizzled boxes of 64 rows x 64 columns) and of one mask box per item; a second lane copies the
//     step's x columns (and col-axis scales), which a small kernel launched just before has written to the
//     workspace in sorted order and in the pair layout described below.  The main kernel is a programmatic
//     dependent of that small kernel: it starts streaming weights at once and only the lane that copies x waits.
//   - Twelve consumer warps: warp = row tile (4) + 4 * item third (3).  A warp owns the accumulators of its up to
//     six items for its 16 rows and walks the four 32-column blocks of a step; inside a block its six items are
//     six independent chains of four dependent MMAs, issued round-robin.  That interleaving is what the speed
//     hangs on: a dependent mma.sync waits ~100 clocks for its accumulator on this GPU, so an SM sub-partition
//     needs many chains in flight (3 warps x 6) to keep its tensor pipe fed.  What bounds the kernel in the end
//     is that pipe: warp-level MMAs run at a quarter of the tcgen05 rate (one m16n8k16 per ~16 clocks and
//     sub-partition), and 16 variants with ~4 tokens each need 2 x 16 of them per 16 rows x 16 columns.
//
// Pair layout.  Inside a block of 32 columns a 32-bit MMA register holds columns (a, a + 16) instead of
// (a, a + 1): then `mask_word << (15 - a)` puts the two sign bits of the pair on bits 15 and 31, and one shift
// plus one LOP3 per register turns mask bits into +-v.  x is laid out that way so that ldmatrix delivers B
// fragments directly; W_b fragments are loaded in natural order (ldmatrix from the swizzled TMA tile) and
// re-paired with eight byte permutes per block, shared by all items.
//
// Batches with more than 18 items run as several passes over the CTA's slice (W_b then comes from L2).
#include <cooperative_groups.h>

#include "pd_ptx.cuh"

namespace cg = cooperative_groups;

namespace pd {
namespace {

constexpr int kMvRows = 64;          // output rows per CTA
constexpr int kMvStepK = 128;        // columns per ring step
constexpr int kMvMaxTokens = 64;     // token rows per launch
constexpr int kMvThirds = 3;         // the items of a pass are dealt to three groups of warps
constexpr int kMvMine = 6;           // items per warp
constexpr int kMvItems = kMvThirds * kMvMine;  // items per pass
constexpr int kMvConsumers = 4 * kMvThirds;
constexpr int kMvThreads = (kMvConsumers + 2) * 32;  // + the weight producer and the x loader
constexpr int kMvPrepThreads = 256;
constexpr int kMvStages = 3;
constexpr int kMvMaxItemsTotal = kMvMaxTokens;  // every item holds at least one token
constexpr int kMvMaxBuckets = 65;               // 64 variants + "base only"

// one ring stage
constexpr int kMvOffW = 0;                                        // 2 boxes [64 rows][128 B], 128-byte swizzle
constexpr int kMvOffMask = 2 * kMvRows * 128;                     // [item][64 rows][4 words]
constexpr int kMvOffX = kMvOffMask + kMvItems * kMvRows * 16;     // [block 4][chunk 4][sorted token m_pad][16 B]
constexpr int kMvOffV = kMvOffX + 4 * 4 * kMvMaxTokens * 16;      // [item][block 4][t 4][16 B] col-axis scale pairs
constexpr int kMvStageBytes = (kMvOffV + kMvItems * 256 + 1023) / 1024 * 1024;  // stages start 1024-byte aligned (swizzle)
// The partial sums [token slot 168][68] fp32 reuse the ring once it has drained.
constexpr int kMvPartStride = 68;    // floats per token slot: 64 rows + padding that spreads the lanes over the banks
constexpr int kMvOffPart = 0;
static_assert(kMvItems * 8 * kMvPartStride * 4 <= kMvStages * kMvStageBytes, "partial sums fit the ring");
constexpr int kMvOffMag = kMvStages * kMvStageBytes;              // [item][64 rows] (v, v) row-axis scales
constexpr int kMvOffRowOff = kMvOffMag + kMvItems * kMvRows * 4;  // [item][lane] ldmatrix row offsets
constexpr int kMvOffTables = kMvOffRowOff + kMvItems * 32 * 4;
struct MvSort {
    int ids[kMvMaxTokens];                  // bucket of token i (V = base only, -2 = not a valid row)
    int tok[kMvMaxTokens];                  // sorted position -> token row
    int cnt[kMvMaxBuckets + 1], start[kMvMaxBuckets + 1], istart[kMvMaxBuckets + 1];  // per bucket: rows, first position, first item
    int item_var[kMvMaxItemsTotal];         // variant (V = base only)
    int item_first[kMvMaxItemsTotal];       // first sorted position
    int item_cnt[kMvMaxItemsTotal];         // tokens (1..8)
    int n_items, n_valid;
};
struct MvTables {
    uint64_t full[kMvStages], empty[kMvStages];
    MvSort sort;
    int abort_flag;
};
constexpr int kMvSmemBytes = kMvOffTables + static_cast<int>(sizeof(MvTables)) + 1024 /* alignment slack */;
static_assert(kMvSmemBytes <= 227 * 1024, "shared memory per CTA");

struct MvArgs {
    const __half *x;
    const int32_t *ids;
    const __half *vs;
    __half *y;
    int64_t ldx, ldy, v_stride;
    unsigned long long col_axis_bits;
    int M, V, d_out, d_in;
    int steps_total;  // d_in / 128
    int m_pad;        // M rounded up to 8: sorted-token rows per chunk of x_pairs
    // written by mv_prepare_kernel, read by mv_decode_kernel:
    //   x_pairs [step][block 4][chunk 4][sorted token m_pad][16 B], v_pairs [variant][step][block 4][t 4][16 B]
    unsigned char *x_pairs;
    unsigned char *v_pairs;
    uint32_t *status;
};

// Buckets the token rows by variant id (stable) and cuts the buckets into items of at most 8 rows.  Called by all
// threads of a CTA (at least kMvMaxBuckets of them); every CTA of both kernels computes the same tables.
__device__ __forceinline__ void mv_sort_rows(MvSort &so, const MvArgs &a, bool report_bad_ids) {
    const int tid = threadIdx.x;
    int my_bucket = -2;
    if (tid < kMvMaxTokens) {
        if (tid < a.M) {
            const int id = a.ids[tid];
            if (id < -1 || id >= a.V) {
                if (report_bad_ids) latch_error(a.status, PD_ERR_BAD_VARIANT, tid);
            } else {
                my_bucket = id < 0 ? a.V : id;
            }
        }
        so.ids[tid] = my_bucket;
    }
    __syncthreads();
    int rank = 0;  // earlier rows of my bucket
    if (tid < a.M && my_bucket >= 0)
        for (int j = 0; j < tid; ++j) rank += so.ids[j] == my_bucket ? 1 : 0;
    if (tid <= a.V) {  // thread b counts bucket b
        int c = 0;
        for (int j = 0; j < a.M; ++j) c += so.ids[j] == tid ? 1 : 0;
        so.cnt[tid] = c;
    }
    __syncthreads();
    if (tid <= a.V + 1) {  // first position and first item of bucket b (entry V + 1: the totals)
        int p = 0, it = 0;
        for (int b = 0; b < tid; ++b) {
            const int c = so.cnt[b];
            p += c;
            it += (c + 7) >> 3;
        }
        so.start[tid] = p;
        so.istart[tid] = it;
        if (tid == a.V + 1) so.n_valid = p, so.n_items = it;
    }
    __syncthreads();
    if (tid < a.M && my_bucket >= 0) {
        const int pos = so.start[my_bucket] + rank;
        so.tok[pos] = tid;
        if ((rank & 7) == 0) {
            const int it = so.istart[my_bucket] + (rank >> 3);
            so.item_var[it] = my_bucket;
            so.item_first[it] = pos;
            so.item_cnt[it] = min(8, so.cnt[my_bucket] - rank);
        }
    }
    __syncthreads();
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 ldg_nc(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void tma_load_4d(const CUtensorMap *map, uint64_t *bar, void *dst, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void mv_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void mv_grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// One CTA per step of 128 columns: the step's x columns of every valid token row, in sorted order and pair layout
// (chunk c of a 32-column block holds, for t = 0..3, the pairs (2t, 2t+16), (2t+8, 2t+24), (2t+1, 2t+17),
// (2t+9, 2t+25) for c = 0..3), and the step's scales of every col-axis variant as pairs
// {(2t, 2t+16), (2t+1, 2t+17), (2t+8, 2t+24), (2t+9, 2t+25)} per (block, t).
template <bool BF16>
__global__ void __launch_bounds__(kMvPrepThreads) mv_prepare_kernel(const MvArgs a) {
    __shared__ MvSort so;
    mv_grid_launch_dependents();  // the decode kernel may start streaming weights; it waits for this grid before it reads x_pairs
    mv_sort_rows(so, a, false);
    const int s = blockIdx.x, k0 = s * kMvStepK;
    const int n_valid = so.n_valid;
    for (int u = threadIdx.x; u < n_valid * 4; u += kMvPrepThreads) {
        const int blk = u / n_valid, pos = u - blk * n_valid;
        const __half *src = a.x + static_cast<size_t>(so.tok[pos]) * a.ldx + k0 + 32 * blk;
        const uint4 l0 = ldg_nc(src), l1 = ldg_nc(src + 8), l2 = ldg_nc(src + 16), l3 = ldg_nc(src + 24);
        const uint32_t x0[4] = {l0.x, l0.y, l0.z, l0.w}, x1[4] = {l1.x, l1.y, l1.z, l1.w};
        const uint32_t x2[4] = {l2.x, l2.y, l2.z, l2.w}, x3[4] = {l3.x, l3.y, l3.z, l3.w};
        uint32_t c[4][4];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            c[0][t] = prmt(x0[t], x2[t], 0x5410u);
            c[2][t] = prmt(x0[t], x2[t], 0x7632u);
            c[1][t] = prmt(x1[t], x3[t], 0x5410u);
            c[3][t] = prmt(x1[t], x3[t], 0x7632u);
        }
        unsigned char *dst = a.x_pairs + static_cast<size_t>(s) * (256 * a.m_pad);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch)
            *reinterpret_cast<uint4 *>(dst + ((blk * 4 + ch) * a.m_pad + pos) * 16) = make_uint4(c[ch][0], c[ch][1], c[ch][2], c[ch][3]);
    }
    if (a.col_axis_bits) {
        for (int u = threadIdx.x; u < a.V * 16; u += kMvPrepThreads) {
            const int var = u >> 4, blk = (u >> 2) & 3, t = u & 3;
            if (!((a.col_axis_bits >> var) & 1ull)) continue;
            const uint32_t *vw = reinterpret_cast<const uint32_t *>(a.vs + static_cast<size_t>(var) * a.v_stride + k0 + 32 * blk);
            const uint32_t w0 = __ldg(vw + t), w1 = __ldg(vw + t + 4), w2 = __ldg(vw + t + 8), w3 = __ldg(vw + t + 12);
            // binary16 scales -> the weights' type (one rounding for bfloat16)
            *reinterpret_cast<uint4 *>(a.v_pairs + (static_cast<size_t>(var) * a.steps_total + s) * 256 + blk * 64 + t * 16) =
                make_uint4(Elem<BF16>::scale_pair2(prmt(w0, w2, 0x5410u)), Elem<BF16>::scale_pair2(prmt(w0, w2, 0x7632u)),
                           Elem<BF16>::scale_pair2(prmt(w1, w3, 0x5410u)), Elem<BF16>::scale_pair2(prmt(w1, w3, 0x7632u)));
        }
    }
}

// ANYCOL: some variant of the call scales along d_in (its items read their scale pairs from the stage).
template <bool BF16, bool ANYCOL>
__global__ void __launch_bounds__(kMvThreads, 1)
mv_decode_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_m, const MvArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    MvTables &tb = *reinterpret_cast<MvTables *>(smem + kMvOffTables);
    float *part = reinterpret_cast<float *>(smem + kMvOffPart);
    uint32_t *mag2 = reinterpret_cast<uint32_t *>(smem + kMvOffMag);
    uint32_t *rowoff = reinterpret_cast<uint32_t *>(smem + kMvOffRowOff);
    volatile int *abort_flag = &tb.abort_flag;

    cg::cluster_group cluster = cg::this_cluster();
    const int n_rank = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = blockIdx.y * kMvRows;
    const int step0 = static_cast<int>((static_cast<int64_t>(rank) * a.steps_total) / n_rank);
    const int step1 = static_cast<int>((static_cast<int64_t>(rank + 1) * a.steps_total) / n_rank);
    const bool is_producer = warp == kMvConsumers && lane == 0;
    constexpr uint32_t kWBytes = 2u * kMvRows * 128u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMvStages; ++s) {
            mbar_init(tb.full + s, 3);  // W_b, masks (producer) and x (loader)
            mbar_init(tb.empty + s, kMvConsumers);
        }
        tb.abort_flag = 0;
        mbar_fence_init();
    }
    mv_grid_launch_dependents();
    // No grid-dependency wait here: this grid is a programmatic dependent of mv_prepare_kernel, which was launched
    // in stream order, so everything older than that kernel is complete.  Only its own output (x_pairs, v_pairs)
    // needs the wait, and only the loader lane reads it.
    __syncthreads();
    int w_issued = 0;  // producer: W_b tiles already requested (the first ring fill goes out before the rows are sorted)
    if (is_producer) {
        prefetch_tensormap(&map_w);
        prefetch_tensormap(&map_m);
        for (int s = step0; s < step1 && w_issued < kMvStages; ++s, ++w_issued) {
            unsigned char *base = smem + w_issued * kMvStageBytes;
            mbar_arrive_expect_tx(tb.full + w_issued, kWBytes);
            tma_load_2d(&map_w, tb.full + w_issued, base + kMvOffW, s * kMvStepK, row0);
            tma_load_2d(&map_w, tb.full + w_issued, base + kMvOffW + kMvRows * 128, s * kMvStepK + 64, row0);
        }
    }
    MvSort &so = tb.sort;
    mv_sort_rows(so, a, blockIdx.x == 0 && blockIdx.y == 0);
    const int n_items_total = so.n_items;
    const int n_pass = (n_items_total + kMvItems - 1) / kMvItems;

    uint32_t gs = 0;  // ring steps so far (every role counts them the same way)
    bool ok = true;

    for (int pass = 0; pass < n_pass; ++pass) {
        const int item0 = pass * kMvItems;
        const int n_it = min(kMvItems, n_items_total - item0);
        // per-pass tables, padded to the full item count with copies of the last item (their sums are never stored):
        // row-axis scales (v, v) per item and row, ldmatrix row offsets per item and lane
        for (int i = threadIdx.x; i < kMvItems * kMvRows; i += kMvThreads) {
            const int it = i / kMvRows, r = i - it * kMvRows;
            uint32_t pair = 0;  // base-only items, col-axis items and padding: +-0
            if (it < n_it) {
                const int var = so.item_var[item0 + it];
                if (var < a.V && !((a.col_axis_bits >> var) & 1ull) && row0 + r < a.d_out)
                    pair = Elem<BF16>::scale_pair(*reinterpret_cast<const unsigned short *>(a.vs + static_cast<size_t>(var) * a.v_stride + row0 + r));
            }
            mag2[i] = pair;
        }
        for (int i = threadIdx.x; i < kMvItems * 32; i += kMvThreads) {
            const int it = min(i >> 5, n_it - 1), l = i & 31;
            const int first = so.item_first[item0 + it], cnt = so.item_cnt[item0 + it];
            // rows past the item's tokens re-read its last token: their output columns are never stored
            rowoff[i] = static_cast<uint32_t>(((l >> 3) * a.m_pad + first + min(l & 7, cnt - 1)) * 16);
        }
        uint32_t delta_bits = 0, col_bits = 0;  // per item of this pass
        for (int it = 0; it < n_it; ++it) {
            const int var = so.item_var[item0 + it];
            if (var < a.V) {
                delta_bits |= 1u << it;
                if ((a.col_axis_bits >> var) & 1ull) col_bits |= 1u << it;
            }
        }
        __syncthreads();

        if (warp == kMvConsumers) {
            // ------------------------------------------------ producer: W_b tile and one mask box per item
            if (lane == 0) {
                const uint32_t mask_tx = static_cast<uint32_t>(__popc(delta_bits)) * kMvRows * 16u;
                for (int s = step0; s < step1; ++s, ++gs) {
                    const int st = gs % kMvStages;
                    unsigned char *base = smem + st * kMvStageBytes;
                    if (w_issued > 0) {
                        --w_issued;  // this stage's W_b tile is already on its way
                    } else {
                        if (!(ok = mbar_wait(tb.empty + st, ((gs / kMvStages) & 1) ^ 1, abort_flag, a.status, 21))) break;
                        mbar_arrive_expect_tx(tb.full + st, kWBytes);
                        tma_load_2d(&map_w, tb.full + st, base + kMvOffW, s * kMvStepK, row0);
                        tma_load_2d(&map_w, tb.full + st, base + kMvOffW + kMvRows * 128, s * kMvStepK + 64, row0);
                    }
                    mbar_arrive_expect_tx(tb.full + st, mask_tx);
                    for (int it = 0; it < n_it; ++it)
                        if ((delta_bits >> it) & 1u)
                            tma_load_4d(&map_m, tb.full + st, base + kMvOffMask + it * (kMvRows * 16), 0, row0, s,
                                        so.item_var[item0 + it]);
                }
            }
        } else if (warp == kMvConsumers + 1) {
            // ------------------------------------------------ x loader: the step's slab of x_pairs and the col-axis scale pairs
            if (lane == 0) {
                if (pass == 0) mv_grid_dependency_wait();  // mv_prepare_kernel has written them
                const uint32_t x_bytes = 256u * static_cast<uint32_t>(a.m_pad);
                const uint32_t tx = x_bytes + static_cast<uint32_t>(__popc(col_bits)) * 256u;
                for (int s = step0; s < step1; ++s, ++gs) {
                    const int st = gs % kMvStages;
                    if (gs >= kMvStages && !(ok = mbar_wait(tb.empty + st, ((gs / kMvStages) & 1) ^ 1, abort_flag, a.status, 22)))
                        break;
                    unsigned char *base = smem + st * kMvStageBytes;
                    mbar_arrive_expect_tx(tb.full + st, tx);
                    bulk_load_1d(base + kMvOffX, a.x_pairs + static_cast<size_t>(s) * x_bytes, x_bytes, tb.full + st);
                    for (int it = 0; it < n_it; ++it)
                        if ((col_bits >> it) & 1u)
                            bulk_load_1d(base + kMvOffV + it * 256,
                                         a.v_pairs + (static_cast<size_t>(so.item_var[item0 + it]) * a.steps_total + s) * 256, 256u,
                                         tb.full + st);
                }
            }
        } else {
            // ------------------------------------------------ consumers: warp = row tile + 4 * item third
            const int g = lane >> 2, t = lane & 3;
            const int rt = warp & 3, third = warp >> 2;  // this warp's items: third, third + 3, third + 6, ...
            float acc[kMvMine][4];
#pragma unroll
            for (int j = 0; j < kMvMine; ++j)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
            // ldmatrix row addresses of the W_b fragments inside a box: matrices (rows 0-7, chunk c), (rows 8-15, c),
            // (rows 0-7, c + 1), (rows 8-15, c + 1); chunk index XORed with the row's low bits (128-byte swizzle)
            const int wrow = rt * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
            uint32_t woff[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) woff[q] = static_cast<uint32_t>(kMvOffW + wrow * 128 + (((2 * q + (lane >> 4)) ^ (wrow & 7)) << 4));
            // `word * mul3` = `word << (6 - 2t)`; the other three alignments are constant shifts of it
            const uint32_t mul3 = 1u << (6 - 2 * t);
            const uint32_t smem_base = smem_u32(smem);
            // per-lane addresses with this warp's first item folded in; item third + 3j adds 3j item strides
            const uint32_t mag_addr = smem_u32(mag2) + static_cast<uint32_t>((third * kMvRows + rt * 16 + g) * 4);
            const uint32_t rowoff_addr = smem_u32(rowoff) + static_cast<uint32_t>((third * 32 + lane) * 4);
            const uint32_t moff = static_cast<uint32_t>(kMvOffMask + third * (kMvRows * 16) + (rt * 16 + g) * 16);
            const uint32_t voff = static_cast<uint32_t>(kMvOffV + third * 256 + t * 16);
            const uint32_t xblk_bytes = 64u * static_cast<uint32_t>(a.m_pad);  // one block of 32 columns: 4 chunks x m_pad rows x 16 B
            const uint32_t my_col_bits = col_bits >> third;
            // row offsets and row-axis scales of this warp's items do not change during the pass
            uint32_t xo[kMvMine], mg[kMvMine], mg8[kMvMine];
#pragma unroll
            for (int j = 0; j < kMvMine; ++j) {
                xo[j] = lds32(rowoff_addr + 3 * j * 128);
                mg[j] = lds32(mag_addr + 3 * j * (kMvRows * 4));
                mg8[j] = lds32(mag_addr + 3 * j * (kMvRows * 4) + 32);
            }
            const int n_mine = (n_it - third + kMvThirds - 1) / kMvThirds;  // items of this warp that exist

            for (int s = step0; s < step1; ++s, ++gs) {
                const int st = gs % kMvStages;
                if (!(ok = __all_sync(0xffffffffu, mbar_wait(tb.full + st, (gs / kMvStages) & 1, abort_flag, a.status, 23)))) break;
                const uint32_t stage = smem_base + st * kMvStageBytes;
                if (n_mine > 0) {
#pragma unroll 1
                    for (int blk = 0; blk < 4; ++blk) {
                        // W_b fragments of the block, re-paired: ab[mma][register]
                        uint32_t ab[2][4];
                        {
                            uint32_t lo[4], hi[4];  // words t, t+4 of rows g / g+8 (columns 0..15), words t+8, t+12 (columns 16..31)
                            const uint32_t wb = stage + (blk >> 1) * (kMvRows * 128);
                            ldmatrix_x4(lo, wb + ((blk & 1) ? woff[2] : woff[0]));
                            ldmatrix_x4(hi, wb + ((blk & 1) ? woff[3] : woff[1]));
                            ab[0][0] = prmt(lo[0], hi[0], 0x5410u), ab[1][0] = prmt(lo[0], hi[0], 0x7632u);  // row g:   (2t, 2t+16), (2t+1, 2t+17)
                            ab[0][1] = prmt(lo[1], hi[1], 0x5410u), ab[1][1] = prmt(lo[1], hi[1], 0x7632u);  // row g+8
                            ab[0][2] = prmt(lo[2], hi[2], 0x5410u), ab[1][2] = prmt(lo[2], hi[2], 0x7632u);  // row g:   (2t+8, 2t+24), (2t+9, 2t+25)
                            ab[0][3] = prmt(lo[3], hi[3], 0x5410u), ab[1][3] = prmt(lo[3], hi[3], 0x7632u);  // row g+8
                        }
                        // The body is branch-free over the warp's items (missing ones repeat the last item and are
                        // dropped at the end): independent accumulator chains, issued round-robin.
                        uint32_t xb[kMvMine][4], m[kMvMine], m8[kMvMine];
                        uint4 vp[kMvMine];
                        const uint32_t xs = stage + kMvOffX + blk * xblk_bytes;
#pragma unroll
                        for (int j = 0; j < kMvMine; ++j) {
                            ldmatrix_x4(xb[j], xs + xo[j]);
                            m[j] = lds32(stage + moff + 3 * j * (kMvRows * 16) + blk * 4);
                            m8[j] = lds32(stage + moff + 3 * j * (kMvRows * 16) + 128 + blk * 4);
                            if (ANYCOL) vp[j] = lds128(stage + voff + 3 * j * 256 + blk * 64);
                        }
#pragma unroll
                        for (int j = 0; j < kMvMine; ++j) Elem<BF16>::mma16816(acc[j], ab[0][0], ab[0][1], ab[0][2], ab[0][3], xb[j][0], xb[j][1]);
#pragma unroll
                        for (int j = 0; j < kMvMine; ++j) Elem<BF16>::mma16816(acc[j], ab[1][0], ab[1][1], ab[1][2], ab[1][3], xb[j][2], xb[j][3]);
                        // +-v from the mask bits: a set bit keeps +v, a clear bit flips the sign
#pragma unroll
                        for (int j = 0; j < kMvMine; ++j) {
                            uint32_t q0 = mg[j], q2 = mg[j], r0 = mg8[j], r2 = mg8[j];
                            if (ANYCOL && ((my_col_bits >> (3 * j)) & 1u)) q0 = r0 = vp[j].x, q2 = r2 = vp[j].z;
                            const uint32_t a3 = m[j] * mul3, b3 = m8[j] * mul3;  // bits 2t+9, 2t+25 on bits 15, 31
                            const uint32_t s0 = lop3_andn_xor(a3 << 9, 0x80008000u, q0), s2 = lop3_andn_xor(a3 << 1, 0x80008000u, q2);
                            const uint32_t u0 = lop3_andn_xor(b3 << 9, 0x80008000u, r0), u2 = lop3_andn_xor(b3 << 1, 0x80008000u, r2);
                            Elem<BF16>::mma16816(acc[j], s0, u0, s2, u2, xb[j][0], xb[j][1]);
                        }
#pragma unroll
                        for (int j = 0; j < kMvMine; ++j) {
                            uint32_t q1 = mg[j], q3 = mg[j], r1 = mg8[j], r3 = mg8[j];
                            if (ANYCOL && ((my_col_bits >> (3 * j)) & 1u)) q1 = r1 = vp[j].y, q3 = r3 = vp[j].w;
                            const uint32_t a3 = m[j] * mul3, b3 = m8[j] * mul3;
                            const uint32_t s1 = lop3_andn_xor(a3 << 8, 0x80008000u, q1), s3 = lop3_andn_xor(a3, 0x80008000u, q3);
                            const uint32_t u1 = lop3_andn_xor(b3 << 8, 0x80008000u, r1), u3 = lop3_andn_xor(b3, 0x80008000u, r3);
                            Elem<BF16>::mma16816(acc[j], s1, u1, s3, u3, xb[j][2], xb[j][3]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(tb.empty + st);
            }

            // ---- sums -> shared memory (over the ring, which has drained once every consumer is here)
            const uint32_t give_up = static_cast<uint32_t>(!ok || *abort_flag);
            uint32_t gave_up;
            asm volatile(
                "{\n"
                ".reg .pred p, q;\n"
                "setp.ne.u32 q, %1, 0;\n"
                "bar.red.or.pred p, 1, %2, q;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(gave_up)
                : "r"(give_up), "n"(kMvConsumers * 32)
                : "memory");
            if (!gave_up) {
                // token slots 2t, 2t+1 of item `third`; rows g, g+8 of this warp's row tile
                float *mine = part + (third * 8 + 2 * t) * kMvPartStride + rt * 16 + g;
#pragma unroll
                for (int j = 0; j < kMvMine; ++j) {
                    if (j < n_mine) {
                        float *p = mine + 3 * j * 8 * kMvPartStride;
                        p[0] = acc[j][0], p[kMvPartStride] = acc[j][1], p[8] = acc[j][2], p[kMvPartStride + 8] = acc[j][3];
                    }
                }
            }
        }

        // ------------------------------------------------ partial sums of the cluster's column slices, in rank order
        cluster.sync();
        if (!*abort_flag) {
            const int total = n_it * 8 * 32;  // (token slot, pair of rows)
            for (int idx = rank * kMvThreads + threadIdx.x; idx < total; idx += n_rank * kMvThreads) {
                const int slot = idx >> 5, rp = idx & 31;
                const int it = slot >> 3, j = slot & 7;
                if (j >= so.item_cnt[item0 + it]) continue;
                float2 sum = make_float2(0.f, 0.f);
                for (int q = 0; q < n_rank; ++q) {
                    const float2 v = *reinterpret_cast<const float2 *>(cluster.map_shared_rank(part, q) + slot * kMvPartStride + 2 * rp);
                    sum.x += v.x, sum.y += v.y;
                }
                const int o = row0 + 2 * rp;
                __half *dst = a.y + static_cast<size_t>(so.tok[so.item_first[item0 + it] + j]) * a.ldy + o;
                unsigned short *out = reinterpret_cast<unsigned short *>(dst);
                if (o < a.d_out) out[0] = Elem<BF16>::from_float(sum.x);
                if (o + 1 < a.d_out) out[1] = Elem<BF16>::from_float(sum.y);
            }
        }
        cluster.sync();  // nobody refills the ring (next pass) or leaves while another rank still reads its sums
    }

    if (n_pass == 0 && is_producer) {
        // no valid row at all: the W_b tiles requested before the sort must land before the shared memory is released
        for (int st = 0; st < w_issued; ++st) {
            mbar_arrive(tb.full + st);
            mbar_arrive(tb.full + st);
            mbar_wait(tb.full + st, 0, abort_flag, a.status, 24);
        }
    }
    if (*abort_flag) {
        // a wait ran out: give copies that may still be in flight time to land before the shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(10000);
    }
}

}  // namespace

size_t mv_decode_scratch_bytes(int64_t M, int32_t V, int64_t d_in) {
    const size_t m_pad = static_cast<size_t>((M + 7) / 8 * 8);
    return round_up(static_cast<size_t>(d_in) * 2 * m_pad, 256) + round_up(static_cast<size_t>(V) * d_in * 2, 256);
}

// M <= 64 token rows with one variant id each, d_in a multiple of 128.  scratch: mv_decode_scratch_bytes() bytes,
// 256-byte aligned.
pd_status launch_mv_decode(const __half *x, int M, int64_t ldx, const int32_t *ids, const __half *w_b, const uint32_t *masks,
                           int64_t mask_stride, const __half *vs, int64_t v_stride, unsigned long long col_axis_bits, int V,
                           int64_t d_out, int64_t d_in, __half *y, int64_t ldy, unsigned char *scratch, uint32_t *status,
                           bool bf16, cudaStream_t stream) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return PD_ERR_CUDA;
    CUtensorMap mw, mm;
    if (!make_map_2d(&mw, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, w_b, d_out, d_in, d_in * 2, 64, kMvRows, CU_TENSOR_MAP_SWIZZLE_128B))
        return PD_ERR_CUDA;
    {
        // masks [V, d_out, d_in/32] seen as {4 words, rows, groups of 128 columns, variant}
        const cuuint64_t dims[4] = {4, static_cast<cuuint64_t>(d_out), static_cast<cuuint64_t>(d_in / 128), static_cast<cuuint64_t>(V)};
        const cuuint64_t strides[3] = {static_cast<cuuint64_t>(d_in / 8), 16, static_cast<cuuint64_t>(mask_stride) * 4};
        const cuuint32_t box[4] = {4, static_cast<cuuint32_t>(kMvRows), 1, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (fn(&mm, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, const_cast<uint32_t *>(masks), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PD_ERR_CUDA;
    }
    MvArgs a;
    a.x = x;
    a.ids = ids;
    a.vs = vs;
    a.y = y;
    a.ldx = ldx;
    a.ldy = ldy;
    a.v_stride = v_stride;
    a.col_axis_bits = col_axis_bits;
    a.M = M;
    a.V = V;
    a.d_out = static_cast<int>(d_out);
    a.d_in = static_cast<int>(d_in);
    a.steps_total = static_cast<int>(d_in / kMvStepK);
    a.m_pad = (M + 7) / 8 * 8;
    a.x_pairs = scratch;
    a.v_pairs = scratch + round_up(static_cast<size_t>(d_in) * 2 * a.m_pad, 256);
    a.status = status;
    if (bf16) mv_prepare_kernel<true><<<a.steps_total, kMvPrepThreads, 0, stream>>>(a);
    else mv_prepare_kernel<false><<<a.steps_total, kMvPrepThreads, 0, stream>>>(a);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return PD_ERR_CUDA;
    // column split: the cluster size (<= 8) whose grid fills the SMs best, counting a fixed cost of about three
    // steps per CTA (sorting, filling the ring, adding up) on top of its share of the steps
    const int row_groups = static_cast<int>((d_out + kMvRows - 1) / kMvRows);
    const int sms = sm_count();
    int best = 1;
    double best_cost = 0;
    for (int ks = 1; ks <= 8 && ks <= a.steps_total; ++ks) {
        const int waves = (row_groups * ks + sms - 1) / sms;
        const double cost = waves * ((a.steps_total + ks - 1) / ks + 3.0);
        if (ks == 1 || cost < best_cost) best = ks, best_cost = cost;
    }
    static std::atomic<bool> configured[4][kMaxDevices];
    const bool any_col = col_axis_bits != 0;
    void (*kernel)(CUtensorMap, CUtensorMap, MvArgs) =
        bf16 ? (any_col ? mv_decode_kernel<true, true> : mv_decode_kernel<true, false>)
             : (any_col ? mv_decode_kernel<false, true> : mv_decode_kernel<false, false>);
    if (!ensure_dynamic_smem(kernel, kMvSmemBytes, configured[(bf16 ? 2 : 0) + (any_col ? 1 : 0)])) return PD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(best), static_cast<unsigned>(row_groups));
    cfg.blockDim = dim3(kMvThreads);
    cfg.dynamicSmemBytes = kMvSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(best);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // dependent of mv_prepare_kernel only
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    count_launch();
    return cuda_ok(cudaLaunchKernelEx(&cfg, kernel, mw, mm, a));
}

}  // namespace pd
