// C ABI of the pd library: argument checks, workspace layout, dispatch.  No device memory is
// allocated here; everything runs on the caller's stream.
#include <climits>

#include "pd_ptx.cuh"

namespace pd {
size_t grouped_table_bytes(int64_t M, int32_t V);

namespace {

constexpr int kMaxVariants = 64;
constexpr int kGemvMaxTokens = 16;  // above it one tensor-core launch (64-token tiles) beats several decode passes over W_b
constexpr int kGroupThreads = 1024;

// workspace layout of the linear calls:
//   [0, 256)                status words
//   [256, 256 + 4*(V+2))    group offsets (rounded up to 512 bytes)
//   [768, 768 + 4*M)        row_index
constexpr size_t kOffsetsBytes = 512;

// Stable counting sort of the row indices by variant id, one CTA.  Warp w owns the contiguous rows
// [w*seg, (w+1)*seg): it counts its rows per bucket, the CTA turns the counts into start positions (bucket
// major, warp minor), and every warp places its rows in order.  Bucket V holds the rows with id -1.
__global__ void __launch_bounds__(kGroupThreads)
group_rows_kernel(const int32_t *__restrict__ ids, int M, int V, int *__restrict__ offsets,
                  int *__restrict__ row_index, uint32_t *__restrict__ status, int4 *__restrict__ tile_table,
                  int *__restrict__ n_token_tiles, int token_tile) {
    constexpr int kWarps = kGroupThreads / 32;
    __shared__ int cnt[kWarps][kMaxVariants + 1];  // rows of warp w in bucket g, then that pair's first position
    __shared__ int start[kMaxVariants + 2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    for (int i = threadIdx.x; i < kWarps * (kMaxVariants + 1); i += kGroupThreads) (&cnt[0][0])[i] = 0;
    __syncthreads();
    const int seg = (M + kWarps - 1) / kWarps;
    const int r0 = warp * seg, r1 = min(M, r0 + seg);
    for (int c = r0; c < r1; c += 32) {
        const int i = c + lane;
        int g = -2;  // -2: no row / invalid id
        if (i < r1) {
            const int id = ids[i];
            if (id < -1 || id >= V) latch_error(status, PD_ERR_BAD_VARIANT, static_cast<uint32_t>(i));
            else g = id < 0 ? V : id;
        }
        const unsigned same = __match_any_sync(0xffffffffu, g);
        if (g >= 0 && (same & lt) == 0) cnt[warp][g] += __popc(same);  // lowest lane of each bucket present
        __syncwarp();
    }
    __syncthreads();
    if (threadIdx.x <= V) {  // bucket totals
        int t = 0;
        for (int w = 0; w < kWarps; ++w) t += cnt[w][threadIdx.x];
        start[threadIdx.x + 1] = t;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        start[0] = 0;
        for (int g = 0; g <= V; ++g) start[g + 1] += start[g];
        for (int g = 0; g <= V + 1; ++g) offsets[g] = start[g];
        if (tile_table != nullptr) {  // cut every bucket into token tiles
            int n = 0;
            for (int g = 0; g <= V; ++g)
                for (int first = start[g]; first < start[g + 1]; first += token_tile)
                    tile_table[n++] = make_int4(g, first, min(token_tile, start[g + 1] - first), 0);
            *n_token_tiles = n;
        }
    }
    __syncthreads();
    if (threadIdx.x <= V) {  // first position of (bucket, warp)
        int pos = start[threadIdx.x];
        for (int w = 0; w < kWarps; ++w) {
            const int c = cnt[w][threadIdx.x];
            cnt[w][threadIdx.x] = pos;
            pos += c;
        }
    }
    __syncthreads();
    for (int c = r0; c < r1; c += 32) {
        const int i = c + lane;
        int g = -2;
        if (i < r1) {
            const int id = ids[i];
            if (id >= -1 && id < V) g = id < 0 ? V : id;
        }
        const unsigned same = __match_any_sync(0xffffffffu, g);
        if (g >= 0) row_index[cnt[warp][g] + __popc(same & lt)] = i;
        __syncwarp();
        if (g >= 0 && (same & lt) == 0) cnt[warp][g] += __popc(same);
        __syncwarp();
    }
}

// x_sorted[i, :] = x[row_index[i], :], 16 bytes per thread.  Only the first *n_valid entries of row_index exist
// (rows with an id outside [-1, V) are in no bucket); the rows of x_sorted past them belong to no token tile.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __half *__restrict__ x, int64_t ldx, const int *__restrict__ n_valid, int vec_per_row,
                   const int *__restrict__ row_index, uint4 *__restrict__ x_sorted) {
    const int64_t total = static_cast<int64_t>(*n_valid) * vec_per_row;
    for (int64_t i = blockIdx.x * 256ll + threadIdx.x; i < total; i += gridDim.x * 256ll) {
        const int r = static_cast<int>(i / vec_per_row), c = static_cast<int>(i - static_cast<int64_t>(r) * vec_per_row);
        x_sorted[i] = *reinterpret_cast<const uint4 *>(x + static_cast<size_t>(row_index[r]) * ldx + 8 * c);
    }
}

// One warp waits, with the library's bounded wait, on an mbarrier that nothing ever arrives on.  The wait gives up
// after limit_cycles, latches PD_ERR_DEVICE_TIMEOUT (detail 99) and the kernel returns normally.
__global__ void bounded_wait_probe_kernel(uint32_t *status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0, &abort_flag, status, 99, limit_cycles);
}

pd_status check_matrix_args(const void *x, int64_t M, int64_t ldx, const void *w_b, int64_t d_out, int64_t d_in,
                            const void *y, int64_t ldy) {
    if (!x || !w_b || !y || M <= 0 || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    if (d_in % 32 != 0 || d_out > INT_MAX / 2 || d_in > INT_MAX / 2 || M > INT_MAX / 2) return PD_ERR_UNSUPPORTED_SHAPE;
    if (ldx < d_in || ldy < d_out) return PD_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_b) || (reinterpret_cast<uintptr_t>(y) & 1u) || ldx % 8 != 0) return PD_ERR_ALIGNMENT;
    return PD_OK;
}

}  // namespace

pd_status launch_group_rows(const int32_t *ids, int M, int V, int *offsets, int *row_index, uint32_t *status,
                            int4 *tile_table, int *n_token_tiles, int token_tile, const __half *x, int64_t ldx,
                            int64_t d_in, __half *x_sorted, cudaStream_t stream) {
    group_rows_kernel<<<1, kGroupThreads, 0, stream>>>(ids, M, V, offsets, row_index, status, tile_table, n_token_tiles,
                                                       token_tile);
    count_launch();
    if (x_sorted != nullptr) {
        const int vec_per_row = static_cast<int>(d_in / 8);
        const int64_t blocks = (static_cast<int64_t>(M) * vec_per_row + 255) / 256;
        gather_rows_kernel<<<static_cast<unsigned>(blocks < 4096 ? blocks : 4096), 256, 0, stream>>>(
            x, ldx, offsets + V + 1, vec_per_row, row_index, reinterpret_cast<uint4 *>(x_sorted));
        count_launch();
    }
    return cuda_ok(cudaGetLastError());
}

// workspace of pd_linear_multivariant beyond the status words, offsets and row index (tensor-core path only)
size_t grouped_table_bytes(int64_t M, int32_t V) {
    const size_t max_tiles = static_cast<size_t>(M / kGroupedMinTokenTile + V + 2);
    return round_up(max_tiles * sizeof(int4), 256) + 256;  // tile table + the tile count
}

}  // namespace pd

using namespace pd;

extern "C" {

size_t pd_workspace_bytes(int op, int64_t M, int32_t V, int64_t d_out, int64_t d_in) {
    switch (op) {
        case PD_OP_PACK:
            return kStatusBytes + pack_scratch_bytes(d_out, d_in);
        case PD_OP_LINEAR:  // + the fp32 partial sums when few tokens make the tensor-core path split its k loop
            return kStatusBytes + ((M > kGemvMaxTokens && d_in >= 64 && d_out > 0) ? gemm_partial_bytes(M, d_out, d_in) : 0);
        case PD_OP_LINEAR_MULTIVARIANT:
            if (M <= 0 || V <= 0) return kStatusBytes + kOffsetsBytes;
            if (M <= kMvDecodeMaxTokens && d_in % 128 == 0)  // decode batches: x (and col-axis scales) re-laid out
                return kStatusBytes + mv_decode_scratch_bytes(M, V, d_in);
            return kStatusBytes + kOffsetsBytes + round_up(sizeof(int) * static_cast<size_t>(M), 256) +
                   (M > kGemvMaxTokens ? grouped_table_bytes(M, V) + round_up(static_cast<size_t>(M) * d_in * 2, 256) : 0);
        case PD_OP_FIT:
            return M > 0 ? kStatusBytes + fit_scratch_bytes(M, d_out, d_in) : 0;
        case PD_OP_FIT_LAYER:
            return M > 0 ? kStatusBytes + fit_layer_scratch_bytes(M, M, d_out, d_in) : 0;
        case PD_OP_MERGE:
        default:
            return 0;
    }
}

const char *pd_status_string(pd_status s) {
    switch (s) {
        case PD_OK: return "ok";
        case PD_ERR_INVALID_ARG: return "invalid argument";
        case PD_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case PD_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
        case PD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case PD_ERR_CUDA: return "CUDA call failed";
        case PD_ERR_BAD_VARIANT: return "variant id out of range";
        case PD_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int64_t pd_launch_count(void) { return g_launches.load(); }

}  // extern "C"

namespace {

pd_status pack_impl(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in, uint32_t *mask, void *v_row,
                    void *v_col, void *workspace, size_t workspace_bytes, void *cuda_stream, bool bf16) {
    if (!w_f || !w_b || !mask || (!v_row && !v_col) || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    if (d_in % 32 != 0 || d_out > INT_MAX / 2 || d_in > INT_MAX / 2) return PD_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(w_f) || !aligned16(w_b) || (reinterpret_cast<uintptr_t>(mask) & 3u)) return PD_ERR_ALIGNMENT;
    if (!workspace || !aligned256(workspace) || workspace_bytes < pd_workspace_bytes(PD_OP_PACK, 0, 0, d_out, d_in))
        return PD_ERR_WORKSPACE;
    auto *sums = reinterpret_cast<unsigned long long *>(static_cast<unsigned char *>(workspace) + kStatusBytes);
    return launch_pack(static_cast<const __half *>(w_f), static_cast<const __half *>(w_b), d_out, d_in, mask,
                       static_cast<__half *>(v_row), static_cast<__half *>(v_col), sums, bf16,
                       static_cast<cudaStream_t>(cuda_stream));
}

pd_status merge_impl(const void *w_b, const uint32_t *mask, const void *v, pd_axis axis, int64_t d_out, int64_t d_in,
                     void *w_hat, void *cuda_stream, bool bf16) {
    if (!w_b || !mask || !v || !w_hat || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    if (axis != PD_AXIS_ROW && axis != PD_AXIS_COL) return PD_ERR_INVALID_ARG;
    if (d_in % 32 != 0 || d_out > INT_MAX / 2 || d_in > INT_MAX / 2) return PD_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(w_b) || !aligned16(w_hat) || (reinterpret_cast<uintptr_t>(mask) & 3u)) return PD_ERR_ALIGNMENT;
    if (axis == PD_AXIS_COL && !aligned16(v)) return PD_ERR_ALIGNMENT;
    return launch_merge(static_cast<const __half *>(w_b), mask, static_cast<const __half *>(v), axis, d_out, d_in,
                        static_cast<__half *>(w_hat), bf16, static_cast<cudaStream_t>(cuda_stream));
}

pd_status linear_impl(const void *x, int64_t M, int64_t ldx, const void *w_b, const uint32_t *mask, const void *v,
                      pd_axis axis, int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace,
                      size_t workspace_bytes, void *cuda_stream, uint32_t flags, bool bf16) {
    pd_status st = check_matrix_args(x, M, ldx, w_b, d_out, d_in, y, ldy);
    if (st != PD_OK) return st;
    if (flags & ~static_cast<uint32_t>(PD_LINEAR_WEIGHTS_RESIDENT)) return PD_ERR_INVALID_ARG;
    if (axis != PD_AXIS_ROW && axis != PD_AXIS_COL) return PD_ERR_INVALID_ARG;
    if (mask && !v) return PD_ERR_INVALID_ARG;
    if (mask && (!aligned16(mask) || !aligned16(v))) return PD_ERR_ALIGNMENT;
    if (!workspace || !aligned256(workspace) || workspace_bytes < pd_workspace_bytes(PD_OP_LINEAR, M, 0, d_out, d_in))
        return PD_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const __half *xh = static_cast<const __half *>(x);
    __half *yh = static_cast<__half *>(y);
    if (M > kGemvMaxTokens && d_in >= 64)  // narrower layers would need a TMA box wider than the matrix
        return launch_gemm(xh, M, ldx, static_cast<const __half *>(w_b), mask, static_cast<const __half *>(v), axis,
                           d_out, d_in, yh, ldy, reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + kStatusBytes),
                           static_cast<uint32_t *>(workspace), bf16, stream);
    GemvScratch scratch;
    scratch.status = static_cast<uint32_t *>(workspace);
    scratch.weights_resident = (flags & PD_LINEAR_WEIGHTS_RESIDENT) != 0;
    scratch.bf16 = bf16;
    for (int64_t m0 = 0; m0 < M; m0 += 16) {
        const int rows = static_cast<int>(M - m0 < 16 ? M - m0 : 16);
        st = launch_gemv(xh + m0 * ldx, rows, ldx, static_cast<const __half *>(w_b), mask,
                         static_cast<const __half *>(v), axis, d_out, d_in, yh + m0 * ldy, ldy, nullptr, nullptr, 0,
                         &scratch, stream);
        if (st != PD_OK) return st;
    }
    return PD_OK;
}

pd_status multivariant_impl(const void *x, int64_t M, int64_t ldx, const int32_t *variant_ids, const void *w_b,
                            const uint32_t *masks, const void *vs, int64_t v_stride, const uint8_t *axes, int32_t V,
                            int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace, size_t workspace_bytes,
                            void *cuda_stream, bool bf16);

}  // namespace

extern "C" {

pd_status pd_pack_delta(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in, uint32_t *mask, void *v_row,
                        void *v_col, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return pack_impl(w_f, w_b, d_out, d_in, mask, v_row, v_col, workspace, workspace_bytes, cuda_stream, false);
}
pd_status pd_pack_delta_bf16(const void *w_f, const void *w_b, int64_t d_out, int64_t d_in, uint32_t *mask, void *v_row,
                             void *v_col, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return pack_impl(w_f, w_b, d_out, d_in, mask, v_row, v_col, workspace, workspace_bytes, cuda_stream, true);
}
pd_status pd_merge(const void *w_b, const uint32_t *mask, const void *v, pd_axis axis, int64_t d_out, int64_t d_in,
                   void *w_hat, void *cuda_stream) {
    return merge_impl(w_b, mask, v, axis, d_out, d_in, w_hat, cuda_stream, false);
}
pd_status pd_merge_bf16(const void *w_b, const uint32_t *mask, const void *v, pd_axis axis, int64_t d_out, int64_t d_in,
                        void *w_hat, void *cuda_stream) {
    return merge_impl(w_b, mask, v, axis, d_out, d_in, w_hat, cuda_stream, true);
}
pd_status pd_linear(const void *x, int64_t M, int64_t ldx, const void *w_b, const uint32_t *mask, const void *v,
                    pd_axis axis, int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace,
                    size_t workspace_bytes, void *cuda_stream) {
    return linear_impl(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, workspace, workspace_bytes, cuda_stream, 0u, false);
}
pd_status pd_linear_ex(const void *x, int64_t M, int64_t ldx, const void *w_b, const uint32_t *mask, const void *v,
                       pd_axis axis, int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace,
                       size_t workspace_bytes, void *cuda_stream, uint32_t flags) {
    return linear_impl(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, workspace, workspace_bytes, cuda_stream, flags, false);
}
pd_status pd_linear_bf16(const void *x, int64_t M, int64_t ldx, const void *w_b, const uint32_t *mask, const void *v,
                         pd_axis axis, int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace,
                         size_t workspace_bytes, void *cuda_stream, uint32_t flags) {
    return linear_impl(x, M, ldx, w_b, mask, v, axis, d_out, d_in, y, ldy, workspace, workspace_bytes, cuda_stream, flags, true);
}
pd_status pd_linear_multivariant(const void *x, int64_t M, int64_t ldx, const int32_t *variant_ids, const void *w_b,
                                 const uint32_t *masks, const void *vs, int64_t v_stride, const uint8_t *axes,
                                 int32_t V, int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace,
                                 size_t workspace_bytes, void *cuda_stream) {
    return multivariant_impl(x, M, ldx, variant_ids, w_b, masks, vs, v_stride, axes, V, d_out, d_in, y, ldy, workspace,
                             workspace_bytes, cuda_stream, false);
}
pd_status pd_linear_multivariant_bf16(const void *x, int64_t M, int64_t ldx, const int32_t *variant_ids, const void *w_b,
                                      const uint32_t *masks, const void *vs, int64_t v_stride, const uint8_t *axes,
                                      int32_t V, int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace,
                                      size_t workspace_bytes, void *cuda_stream) {
    return multivariant_impl(x, M, ldx, variant_ids, w_b, masks, vs, v_stride, axes, V, d_out, d_in, y, ldy, workspace,
                             workspace_bytes, cuda_stream, true);
}

pd_status pd_linear_host(const void *x_host, void *x_dev, int64_t M, const void *w_b, const uint32_t *mask, const void *v,
                         pd_axis axis, int64_t d_out, int64_t d_in, void *y_dev, void *y_host, void *workspace,
                         size_t workspace_bytes, void *cuda_stream, uint32_t flags) {
    if (!x_host || !x_dev || !y_dev || !y_host || M <= 0 || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(x_dev, x_host, static_cast<size_t>(M) * d_in * sizeof(__half), cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return PD_ERR_CUDA;
    const pd_status st = linear_impl(x_dev, M, d_in, w_b, mask, v, axis, d_out, d_in, y_dev, d_out, workspace, workspace_bytes,
                                     cuda_stream, flags, false);
    if (st != PD_OK) return st;
    return cuda_ok(cudaMemcpyAsync(y_host, y_dev, static_cast<size_t>(M) * d_out * sizeof(__half), cudaMemcpyDeviceToHost, stream));
}

}  // extern "C"

namespace {
pd_status multivariant_impl(const void *x, int64_t M, int64_t ldx, const int32_t *variant_ids, const void *w_b,
                            const uint32_t *masks, const void *vs, int64_t v_stride, const uint8_t *axes, int32_t V,
                            int64_t d_out, int64_t d_in, void *y, int64_t ldy, void *workspace, size_t workspace_bytes,
                            void *cuda_stream, bool bf16) {
    pd_status st = check_matrix_args(x, M, ldx, w_b, d_out, d_in, y, ldy);
    if (st != PD_OK) return st;
    if (!variant_ids || !masks || !vs || !axes || V <= 0) return PD_ERR_INVALID_ARG;
    if (V > kMaxVariants) return PD_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(masks) || !aligned16(vs) || v_stride % 8 != 0) return PD_ERR_ALIGNMENT;
    for (int g = 0; g < V; ++g) {
        if (axes[g] != PD_AXIS_ROW && axes[g] != PD_AXIS_COL) return PD_ERR_INVALID_ARG;
        if (v_stride < (axes[g] == PD_AXIS_ROW ? d_out : d_in)) return PD_ERR_INVALID_ARG;
    }
    if (!workspace || !aligned256(workspace) ||
        workspace_bytes < pd_workspace_bytes(PD_OP_LINEAR_MULTIVARIANT, M, V, d_out, d_in))
        return PD_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    auto *base = static_cast<unsigned char *>(workspace);
    auto *status = reinterpret_cast<uint32_t *>(base);
    int *offsets = reinterpret_cast<int *>(base + kStatusBytes);
    int *row_index = reinterpret_cast<int *>(base + kStatusBytes + kOffsetsBytes);
    const __half *xh = static_cast<const __half *>(x);
    const __half *vh = static_cast<const __half *>(vs);
    const int64_t mask_words = d_out * (d_in / 32);
    unsigned long long col_bits = 0;
    for (int g = 0; g < V; ++g)
        if (axes[g] == PD_AXIS_COL) col_bits |= 1ull << g;
    if (M <= kMvDecodeMaxTokens && d_in % 128 == 0)
        // a decode batch: one launch that streams W_b once and applies every variant's mask to its few rows
        return launch_mv_decode(xh, static_cast<int>(M), ldx, variant_ids, static_cast<const __half *>(w_b), masks, mask_words, vh,
                                v_stride, col_bits, V, d_out, d_in, static_cast<__half *>(y), ldy, base + kStatusBytes, status, bf16, stream);
    if (M > kGemvMaxTokens && d_in >= 64) {
        // more than one decode chunk: sort the rows by variant, gather them, one grouped tensor-core launch
        unsigned char *p = base + kStatusBytes + kOffsetsBytes + round_up(sizeof(int) * static_cast<size_t>(M), 256);
        int4 *tile_table = reinterpret_cast<int4 *>(p);
        int *n_token_tiles = reinterpret_cast<int *>(p + grouped_table_bytes(M, V) - 256);
        __half *x_sorted = reinterpret_cast<__half *>(p + grouped_table_bytes(M, V));
        st = launch_group_rows(variant_ids, static_cast<int>(M), V, offsets, row_index, status, tile_table, n_token_tiles,
                               grouped_token_tile_for(M, V, d_out), xh, ldx, d_in, x_sorted, stream);
        if (st != PD_OK) return st;
        return launch_gemm_grouped(x_sorted, M, static_cast<const __half *>(w_b), masks, mask_words, vh, v_stride, col_bits,
                                   V, d_out, d_in, static_cast<__half *>(y), ldy, tile_table, n_token_tiles,
                                   static_cast<int>(M / grouped_token_tile_for(M, V, d_out) + V + 2), grouped_token_tile_for(M, V, d_out), row_index, status,
                                   bf16, stream);
    }
    st = launch_group_rows(variant_ids, static_cast<int>(M), V, offsets, row_index, status, nullptr, nullptr, 0, nullptr, 0, 0,
                           nullptr, stream);
    if (st != PD_OK) return st;
    GemvScratch scratch;
    scratch.status = status;
    scratch.weights_resident = false;
    scratch.bf16 = bf16;
    for (int g = 0; g <= V; ++g) {
        const bool base_only = (g == V);
        st = launch_gemv(xh, 0, ldx, static_cast<const __half *>(w_b), base_only ? nullptr : masks + g * mask_words,
                         base_only ? nullptr : vh + g * v_stride, base_only ? PD_AXIS_ROW : axes[g], d_out, d_in,
                         static_cast<__half *>(y), ldy, row_index, offsets, g, &scratch, stream);
        if (st != PD_OK) return st;
    }
    return PD_OK;
}
}  // namespace

extern "C" {

size_t pd_artifact_bytes(int64_t d_out, int64_t d_in, pd_axis axis) {
    if (d_out <= 0 || d_in <= 0 || d_in % 32 != 0) return 0;
    const size_t mask_bytes = static_cast<size_t>(d_out) * static_cast<size_t>(d_in / 32) * 4;
    return round_up(mask_bytes, 16) + round_up(2 * static_cast<size_t>(axis == PD_AXIS_ROW ? d_out : d_in), 16);
}

pd_status pd_load_merged(const pd_module *modules, int32_t n, void *staging, size_t staging_bytes, void *copy_stream,
                         void *compute_stream) {
    if (!modules || n <= 0 || !staging) return PD_ERR_INVALID_ARG;
    if (!aligned256(staging)) return PD_ERR_ALIGNMENT;
    size_t half = 0;
    for (int i = 0; i < n; ++i) {
        const pd_module &m = modules[i];
        if (!m.w_b || !m.w_hat || !m.artifact || m.d_out <= 0 || m.d_in <= 0) return PD_ERR_INVALID_ARG;
        if ((m.axis != PD_AXIS_ROW && m.axis != PD_AXIS_COL) || (m.bf16 != 0 && m.bf16 != 1)) return PD_ERR_INVALID_ARG;
        if (m.d_in % 32 != 0 || m.d_out > INT_MAX / 2 || m.d_in > INT_MAX / 2) return PD_ERR_UNSUPPORTED_SHAPE;
        if (!aligned16(m.w_b) || !aligned16(m.w_hat)) return PD_ERR_ALIGNMENT;
        const size_t bytes = round_up(pd_artifact_bytes(m.d_out, m.d_in, static_cast<pd_axis>(m.axis)), 256);
        half = bytes > half ? bytes : half;
    }
    if (staging_bytes < 2 * half) return PD_ERR_WORKSPACE;
    cudaStream_t copy = static_cast<cudaStream_t>(copy_stream), compute = static_cast<cudaStream_t>(compute_stream);
    cudaEvent_t copied[2] = {nullptr, nullptr}, merged[2] = {nullptr, nullptr}, start = nullptr;
    pd_status st = PD_OK;
    for (int b = 0; b < 2 && st == PD_OK; ++b)
        if (cudaEventCreateWithFlags(&copied[b], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&merged[b], cudaEventDisableTiming) != cudaSuccess)
            st = PD_ERR_CUDA;
    if (st == PD_OK && cudaEventCreateWithFlags(&start, cudaEventDisableTiming) != cudaSuccess) st = PD_ERR_CUDA;
    // the copies may not start before work queued earlier on the compute stream (which may still read the staging
    // buffer or write the base) has finished
    if (st == PD_OK && (cudaEventRecord(start, compute) != cudaSuccess || cudaStreamWaitEvent(copy, start, 0) != cudaSuccess))
        st = PD_ERR_CUDA;
    for (int i = 0; i < n && st == PD_OK; ++i) {
        const pd_module &m = modules[i];
        const int b = i & 1;
        unsigned char *dst = static_cast<unsigned char *>(staging) + b * half;
        const size_t mask_bytes = round_up(static_cast<size_t>(m.d_out) * static_cast<size_t>(m.d_in / 32) * 4, 16);
        if (i >= 2 && cudaStreamWaitEvent(copy, merged[b], 0) != cudaSuccess) st = PD_ERR_CUDA;  // the half is free again
        if (st == PD_OK && cudaMemcpyAsync(dst, m.artifact, pd_artifact_bytes(m.d_out, m.d_in, static_cast<pd_axis>(m.axis)),
                                           cudaMemcpyHostToDevice, copy) != cudaSuccess)
            st = PD_ERR_CUDA;
        if (st == PD_OK && (cudaEventRecord(copied[b], copy) != cudaSuccess || cudaStreamWaitEvent(compute, copied[b], 0) != cudaSuccess))
            st = PD_ERR_CUDA;
        if (st == PD_OK)
            st = merge_impl(m.w_b, reinterpret_cast<const uint32_t *>(dst), dst + mask_bytes, static_cast<pd_axis>(m.axis), m.d_out,
                            m.d_in, m.w_hat, compute_stream, m.bf16 != 0);
        if (st == PD_OK && cudaEventRecord(merged[b], compute) != cudaSuccess) st = PD_ERR_CUDA;
    }
    for (int b = 0; b < 2; ++b) {  // destroying an event that is still pending only releases it once it has completed
        if (copied[b]) cudaEventDestroy(copied[b]);
        if (merged[b]) cudaEventDestroy(merged[b]);
    }
    if (start) cudaEventDestroy(start);
    return st;
}

static pd_status fit_shape_check(int64_t M, int64_t d_out, int64_t d_in) {
    if (M <= 0 || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    if (d_in % 32 != 0 || d_out % 8 != 0 || M > (1ll << 30) / 128 * 128 || d_out > (1 << 30) || d_in > (1 << 30)) return PD_ERR_UNSUPPORTED_SHAPE;
    return PD_OK;
}

pd_status pd_transpose_mask(const uint32_t *mask, int64_t d_out, int64_t d_in, uint32_t *mask_t, void *cuda_stream) {
    if (!mask || !mask_t || d_out <= 0 || d_in <= 0) return PD_ERR_INVALID_ARG;
    if (d_in % 32 != 0 || (d_out + 31) / 32 > 65535) return PD_ERR_UNSUPPORTED_SHAPE;
    return launch_transpose_mask(mask, d_out, d_in, mask_t, static_cast<cudaStream_t>(cuda_stream));
}

pd_status pd_fit_loss_grad(const void *x, const void *y, int64_t M, const void *w_b, const uint32_t *mask,
                           const uint32_t *mask_t, const float *v, pd_axis axis, int64_t d_out, int64_t d_in, float *loss,
                           float *grad, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!x || !y || !w_b || !mask || !v) return PD_ERR_INVALID_ARG;
    if (axis != PD_AXIS_ROW && axis != PD_AXIS_COL && axis != PD_AXIS_SCALAR) return PD_ERR_INVALID_ARG;
    if (axis == PD_AXIS_COL && grad && !mask_t) return PD_ERR_INVALID_ARG;
    const pd_status shape = fit_shape_check(M, d_out, d_in);
    if (shape != PD_OK) return shape;
    if (!aligned16(x) || !aligned16(y) || !aligned16(w_b)) return PD_ERR_ALIGNMENT;
    if (!workspace || !aligned256(workspace) || workspace_bytes < pd_workspace_bytes(PD_OP_FIT, M, 0, d_out, d_in)) return PD_ERR_WORKSPACE;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    return launch_fit_loss_grad(static_cast<const __half *>(x), static_cast<const __half *>(y), M, static_cast<const __half *>(w_b), mask,
                                mask_t, v, axis, d_out, d_in, loss, grad, ws + kStatusBytes, reinterpret_cast<uint32_t *>(ws),
                                static_cast<cudaStream_t>(cuda_stream));
}

pd_status pd_fit_adamw_step(float *v, float *m1, float *m2, const float *grad, int64_t len, int64_t t, const pd_adamw *opt,
                            void *cuda_stream) {
    if (!v || !m1 || !m2 || !grad || !opt || len <= 0 || t <= 0 || len > (1ll << 31) - 256) return PD_ERR_INVALID_ARG;
    return launch_fit_adamw(v, m1, m2, grad, len, t, opt->lr, opt->beta1, opt->beta2, opt->eps, opt->weight_decay, nullptr,
                            static_cast<cudaStream_t>(cuda_stream));
}

pd_status pd_fit_layer(const void *x_tr, const void *y_tr, int64_t M_tr, const void *x_val, const void *y_val, int64_t M_val,
                       const void *w_b, const uint32_t *mask, const void *v_row0, const void *v_col0, int64_t d_out,
                       int64_t d_in, int32_t epochs, int64_t batch, const pd_adamw *opt, int32_t cosine, void *v_out,
                       int32_t *axis_out, float *val_loss, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!x_tr || !y_tr || !x_val || !y_val || !w_b || !mask || !v_row0 || !v_col0 || !opt || !v_out || !axis_out || !val_loss)
        return PD_ERR_INVALID_ARG;
    if (epochs < 0 || batch <= 0) return PD_ERR_INVALID_ARG;
    pd_status shape = fit_shape_check(M_tr, d_out, d_in);
    if (shape == PD_OK) shape = fit_shape_check(M_val, d_out, d_in);
    if (shape != PD_OK) return shape;
    if ((d_out + 31) / 32 > 65535) return PD_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(x_tr) || !aligned16(x_val) || !aligned16(y_tr) || !aligned16(y_val) || !aligned16(w_b)) return PD_ERR_ALIGNMENT;
    if ((batch * d_out) % 8 != 0 && batch < M_tr) return PD_ERR_ALIGNMENT;  // every minibatch of y starts 16-byte aligned
    if (batch > M_tr) batch = M_tr;
    const int64_t m_max = batch > M_val ? batch : M_val;
    if (!workspace || !aligned256(workspace) || workspace_bytes < pd_workspace_bytes(PD_OP_FIT_LAYER, m_max, 0, d_out, d_in))
        return PD_ERR_WORKSPACE;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    return launch_fit_layer(static_cast<const __half *>(x_tr), static_cast<const __half *>(y_tr), M_tr, static_cast<const __half *>(x_val),
                            static_cast<const __half *>(y_val), M_val, static_cast<const __half *>(w_b), mask,
                            static_cast<const __half *>(v_row0), static_cast<const __half *>(v_col0), d_out, d_in, epochs, batch, *opt,
                            cosine, static_cast<__half *>(v_out), axis_out, val_loss, ws + kStatusBytes,
                            reinterpret_cast<uint32_t *>(ws), static_cast<cudaStream_t>(cuda_stream));
}

pd_status pd_selftest_bounded_wait(void *workspace, int64_t limit_cycles, void *cuda_stream) {
    if (!workspace || !aligned256(workspace) || limit_cycles <= 0 || limit_cycles > 100000000) return PD_ERR_INVALID_ARG;
    bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<uint32_t *>(workspace), limit_cycles);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

pd_status pd_device_status(void *workspace, void *cuda_stream) {
    if (!workspace) return PD_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint32_t words[2] = {0, 0};
    if (cudaMemcpyAsync(words, workspace, sizeof(words), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return PD_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return PD_ERR_CUDA;
    if (words[0] != 0) {
        if (cudaMemsetAsync(workspace, 0, kStatusBytes, stream) != cudaSuccess) return PD_ERR_CUDA;
    }
    return static_cast<pd_status>(words[0]);
}

}  // extern "C"
